"""bfq_dequant_gemm (the dense products of the reconstruction loss, paper Sec. 3.4) against float64 numpy, operand kind
by operand kind.  Tolerances from the arithmetic: integer codes and bf16 numbers are exact operands; an fp32 number is
split into two bf16 terms, relative error <= 2^-17 per element; accumulation is fp32 over K terms.  So for every
output  |c - ref| <= (eA + eB + K 2^-24) sum_k |A(i, k)| |B(j, k)|  with e = 2^-17 for an fp32 operand and 0 otherwise
(+ one fp32 rounding of the result); the tests allow twice that."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_09679_b200 import GemmOperand, Plan, synth
from parity import to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_codes(rows, k, bits, seed):
    """Codes + scales as bfq_forward_quant writes them, from the oracle's quantizer on random rows."""
    y = synth.rows(rows, k, "student_t3", seed, outliers=4, outlier_scale=20.0, dtype=torch.float32)
    codes, scales = oracle.quantize(to_f64(y), bits)
    packed = torch.from_numpy(oracle.pack(codes, bits))
    s16 = torch.from_numpy(scales.view(np.int16)).view(torch.float16)
    return packed, s16, oracle.dequantize(codes, scales)       # dequantized values, float64 [rows][k]


def operand(kind, rows, k, transposed, seed):
    """-> (GemmOperand on the device, float64 [rows][k] values, relative operand error)."""
    if kind in ("f32", "bf16"):
        dt = torch.float32 if kind == "f32" else torch.bfloat16
        v = synth.rows(rows, k, "normal", seed, dtype=dt)
        t = v.t().contiguous() if transposed else v
        return GemmOperand(t.to(DEV), transposed=transposed), to_f64(v), (2.0 ** -17 if kind == "f32" else 0.0)
    bits = int(kind[-1])
    if not transposed:
        packed, s16, val = make_codes(rows, k, bits, seed)
        return GemmOperand(packed.to(DEV), s16.to(DEV), bits), val, 0.0
    packed, s16, val = make_codes(k, rows, bits, seed)          # stored [K][rows]: scales per k
    return GemmOperand(packed.to(DEV), s16.to(DEV), bits, transposed=True), val.T.copy(), 0.0


def check(p, A, a64, ea, B, b64, eb, alpha=1.0):
    c = to_f64(p.dequant_gemm(A, B, alpha))
    ref = alpha * (a64 @ b64.T)
    k = a64.shape[1]
    bound = (ea + eb + (k + 2) * 2.0 ** -24) * abs(alpha) * (np.abs(a64) @ np.abs(b64).T)
    assert c.shape == ref.shape and np.isfinite(c).all()
    worst = (np.abs(c - ref) / np.maximum(2 * bound, 1e-300)).max()
    assert worst <= 1.0, worst
    assert p.device_status() == 0


KINDS = ["f32", "bf16", "codes2", "codes4", "codes8"]


@pytest.mark.parametrize("ka", KINDS)
@pytest.mark.parametrize("kb", KINDS)
@pytest.mark.parametrize("ta,tb", [(False, False), (False, True), (True, True)])
def test_every_operand_kind(ka, kb, ta, tb):
    m, n, k = 200, 136, 192            # ragged tiles in m and n, three K blocks
    # a transposed code operand packs its rows along the stored row: stored rows must stay 16-byte multiples
    if ta and ka.startswith("codes"):
        m = 256 if ka == "codes2" else 224
    if tb and kb.startswith("codes"):
        n = 192 if kb == "codes2" else 160
    p = Plan(256, DEV)
    A, a64, ea = operand(ka, m, k, ta, 900)
    B, b64, eb = operand(kb, n, k, tb, 901)
    check(p, A, a64, ea, B, b64, eb, alpha=0.5)


def test_exact_integer_product_of_two_code_operands():
    """W4A4: both operands codes along K -> an exact integer product times the two scales."""
    p = Plan(256, DEV)
    A, a64, _ = operand("codes4", 300, 4096, False, 910)
    B, b64, _ = operand("codes4", 260, 4096, False, 911)
    c = to_f64(p.dequant_gemm(A, B))
    ref = a64 @ b64.T
    assert np.abs(c - ref).max() <= 2.0 ** -22 * np.abs(ref).max()   # two roundings (scales) of an exact sum


def test_argument_validation():
    from paper_2509_09679_b200 import BfqError
    p = Plan(256, DEV)
    a = GemmOperand(torch.zeros((8, 100), device=DEV))
    b = GemmOperand(torch.zeros((8, 100), device=DEV))
    with pytest.raises(BfqError) as e:
        p.dequant_gemm(a, b)                                      # K not a multiple of 64
    assert e.value.status == -5
    c = p.dequant_gemm(GemmOperand(torch.zeros((0, 64), device=DEV)), GemmOperand(torch.zeros((8, 64), device=DEV)))
    assert c.shape == (0, 8)
