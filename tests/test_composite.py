"""GPU parity of the composite transform Q1 (x) Q2 (paper Sec. 3.3) against the CPU oracle: the Cayley factor, the
unquantized rows and the quantized rows, for several (n1, n2) including the paper's 40 x 128."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_09679_b200 import BfqError, Plan, synth
from parity import check_quant, check_rows_close, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def setup(n1, n2, rows, dtype, seed=3, std=0.1):
    theta2 = synth.angles(n2, "normal", seed)
    params = synth.cayley_params(n1, seed, std)
    x = synth.rows(rows, n1 * n2, "student_t3", seed + 1, outliers=4, outlier_scale=20.0, dtype=dtype)
    p = Plan(n2, DEV)
    p.set_angles(theta2.to(DEV))
    q1 = p.cayley(params.to(DEV), n1)
    Q1_ref = oracle.cayley(to_f64(params), n1)
    return p, q1, Q1_ref, to_f64(theta2), x


@pytest.mark.parametrize("n1", [2, 3, 17, 40, 64])
@pytest.mark.parametrize("std", [0.05, 1.0])
def test_cayley_factor(n1, std):
    params = synth.cayley_params(n1, 11, std)
    p = Plan(128, DEV)
    q1 = to_f64(p.cayley(params.to(DEV), n1))
    ref = oracle.cayley(to_f64(params), n1)
    assert np.abs(q1 - ref).max() <= 2e-7
    assert np.abs(q1 @ q1.T - np.eye(n1)).max() <= 2e-6


@pytest.mark.parametrize("n1,n2,rows", [(3, 16, 7), (5, 64, 130), (12, 256, 33), (40, 128, 61), (64, 256, 9), (7, 1024, 20)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_composite_forward(n1, n2, rows, dtype):
    p, q1, Q1_ref, th2, x = setup(n1, n2, rows, dtype)
    if dtype == torch.bfloat16 and (n1, n2) == (40, 128):
        pytest.skip("covered by the tensor-core tests")
    y_ref = oracle.composite_forward(Q1_ref, th2, to_f64(x))
    amax = np.abs(to_f64(x)).max(axis=1)
    y = p.composite_forward(q1, x.to(DEV), out_dtype=torch.float32)
    check_rows_close(y, y_ref, amax, "composite fp32 out")
    yb = p.composite_forward(q1, x.to(DEV), out_dtype=torch.bfloat16)
    check_rows_close(yb, y_ref, amax, "composite bf16 out")
    assert p.device_status() == 0


@pytest.mark.parametrize("n1,n2,rows", [(3, 16, 7), (12, 256, 33), (40, 128, 61)])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_composite_forward_quant(n1, n2, rows, bits):
    p, q1, Q1_ref, th2, x = setup(n1, n2, rows, torch.float32)
    y_ref = oracle.composite_forward(Q1_ref, th2, to_f64(x))
    codes, scales = p.composite_forward_quant(q1, x.to(DEV), bits)
    check_quant(codes, scales, y_ref, bits, "composite quant")


def test_composite_identity_factor_is_the_butterfly_on_every_run():
    n1, n2, rows = 6, 128, 10
    p, _, _, th2, x = setup(n1, n2, rows, torch.float32)
    eye = torch.eye(n1, dtype=torch.float32, device=DEV)
    y = p.composite_forward(eye, x.to(DEV))
    y_runs = p.forward(x.to(DEV).reshape(rows * n1, n2)).reshape(rows, n1 * n2)
    assert torch.equal(y, y_runs) or (y - y_runs).abs().max() <= 1e-5 * x.abs().max()


def test_composite_argument_validation():
    p = Plan(128, DEV)
    p.set_angles(synth.angles(128, "normal", 1).to(DEV))
    x = torch.zeros((4, 40 * 128), dtype=torch.float32, device=DEV)
    with pytest.raises(BfqError) as e:
        p.composite_forward(torch.eye(65, device=DEV), torch.zeros((1, 65 * 128), device=DEV))
    assert e.value.status == -2
    big = Plan(2048, DEV)
    big.set_angles(synth.angles(2048, "normal", 1).to(DEV))
    with pytest.raises(BfqError) as e:
        big.composite_forward(torch.eye(2, device=DEV), torch.zeros((1, 4096), device=DEV))
    assert e.value.status == -2
    with pytest.raises(BfqError) as e:
        p.composite_forward_quant(torch.eye(40, device=DEV), x, 3)
    assert e.value.status == -3
    fresh = Plan(128, DEV)
    with pytest.raises(BfqError) as e:
        fresh.composite_forward(torch.eye(40, device=DEV), x)
    assert e.value.status == -7
    y = p.composite_forward(torch.eye(40, device=DEV), x[:0])
    assert y.shape == (0, 5120)


# ---- 40 x 128 on bf16 rows: the dense factor runs on the tensor cores in TF32 ------------------------------------
# Tolerance from the arithmetic: both operands of every product are rounded to 11 significant bits (relative error
# 2^-12 each, round to nearest), the accumulation is fp32, so
#     |y - y_ref| <= 2^-11 (1 + 2^-13) sum_k |Q1[i][k]| |X'[k][j]|  +  the fp32 error of the butterfly (1e-5 max|x|).
# The test allows 2^-10 of that sum (twice the bound).
PATHS = ["dense", "butterfly"]


def _select(monkeypatch, path):
    """dense (default): both factors on the tensor cores; butterfly: Q2 as an fp32 butterfly on the CUDA cores."""
    if path == "butterfly":
        monkeypatch.setenv("BFQ_COMPOSITE_FP32_BUTTERFLY", "1")
    else:
        monkeypatch.delenv("BFQ_COMPOSITE_FP32_BUTTERFLY", raising=False)


# The dense path merges the seven stages of Q2 into one 128 x 128 block held as two bf16 terms (relative error 2^-17 per
# entry, the bf16 rows are exact operands) and hands X' to the second product by letting the tensor core read the fp32
# accumulators as TF32, i.e. truncated (relative error up to 2^-10) instead of rounded (2^-12):
#     |y - y_ref| <= (2^-10 + 2^-12) sum_k |Q1||X'|  +  2^-17 sum_k |Q1| (|Q2| |x|).
# The test allows 2^-9 of the first sum and 2^-16 of the second for that path.
def _tf32_setup(rows, seed=5, std=0.1, angle_kind="normal", dist="student_t3", path="butterfly"):
    n1, n2 = 40, 128
    theta2 = synth.angles(n2, angle_kind, seed)
    params = synth.cayley_params(n1, seed, std)
    x = synth.rows(rows, n1 * n2, dist, seed + 1, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    p = Plan(n2, DEV)
    p.set_angles(theta2.to(DEV))
    q1 = p.cayley(params.to(DEV), n1)
    Q1 = oracle.cayley(to_f64(params), n1)
    x64 = to_f64(x)
    inner = oracle.forward(to_f64(theta2), x64.reshape(-1, n2)).reshape(rows, n1, n2)
    y_ref = np.einsum("ik,rkj->rij", Q1, inner).reshape(rows, -1)
    assert np.array_equal(y_ref, oracle.composite_forward(Q1, to_f64(theta2), x64))
    tol = 2.0 ** -10 * np.einsum("ik,rkj->rij", np.abs(Q1), np.abs(inner)).reshape(rows, -1)
    if path == "dense":
        Q2 = oracle.forward(to_f64(theta2), np.eye(n2)).T  # column c = Q2 e_c
        absin = (np.abs(x64).reshape(-1, n2) @ np.abs(Q2).T).reshape(rows, n1, n2)
        tol = 2.0 * tol + 2.0 ** -16 * np.einsum("ik,rkj->rij", np.abs(Q1), absin).reshape(rows, -1)
    tol = tol + 1e-5 * np.abs(x64).max(axis=1, keepdims=True)
    return p, q1, x, y_ref, tol


def _check_tf32_rows(y, y_ref, tol, what):
    o = to_f64(y)
    assert np.isfinite(o).all()
    t = tol + (2.0 ** -8 * np.abs(y_ref) if y.dtype == torch.bfloat16 else 0.0)
    err = np.abs(o - y_ref)
    k = np.unravel_index(np.argmax(err - t), err.shape)
    assert (err <= t).all(), f"{what}: {int((err > t).sum())} out of tolerance; worst at {k}: {err[k]:.3e} > {t[k]:.3e}"


def _check_tf32_quant(codes, scales, y_ref, tol, what, bits=4):
    rows, d = y_ref.shape
    qmax = (1 << (bits - 1)) - 1
    got_codes = oracle.unpack(codes.cpu().numpy(), bits)
    got_s = scales.cpu().view(torch.int16).numpy().view(np.uint16)
    _, ref_s = oracle.quantize(y_ref, bits)
    s_got, s_ref = oracle.f16_bits_to_f64(got_s), oracle.f16_bits_to_f64(ref_s)
    # the absmax moves by at most the tolerance at the extreme element; one fp16 rounding on top
    assert np.all(np.abs(s_got - s_ref) <= tol.max(axis=1) / qmax + 2.0 ** -10 * s_ref + 1e-30), f"{what}: scales"
    ref_codes, _, pre = oracle.quantize(y_ref, bits, scale_in=got_s, want_prequant=True)
    diff = got_codes.astype(np.int32) - ref_codes.astype(np.int32)
    bad = diff != 0
    if bad.any():
        # a code may differ from the oracle's only as far as the element's error bound, in code units, carries the
        # pre-rounding value across rounding boundaries: |code - clip(y_ref / s)| <= 1/2 + tol / s
        allowed = tol / np.maximum(s_got, 1e-30)[:, None] + 1e-4
        dist = np.abs(got_codes.astype(np.float64) - np.clip(pre, -qmax - 1, qmax))
        assert np.all(dist[bad] <= 0.5 + allowed[bad]), f"{what}: code further from the oracle's value than the error bound allows"
        if bits == 4:
            assert np.all(np.abs(diff[bad]) == 1), f"{what}: codes differ by more than one"
    return float(bad.mean())


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("rows", [1, 2, 3, 4, 5, 7, 8, 9, 591, 592, 593, 148 * 8 + 3, 2500])
def test_tensor_core_composite_5120(rows, path, monkeypatch):
    _select(monkeypatch, path)
    p, q1, x, y_ref, tol = _tf32_setup(rows, path=path)
    xd = x.to(DEV)
    y = p.composite_forward(q1, xd)
    assert p.device_status() == 0
    _check_tf32_rows(y, y_ref, tol, "bf16 rows")
    codes, scales = p.composite_forward_quant(q1, xd, 4)
    assert p.device_status() == 0
    frac = _check_tf32_quant(codes, scales, y_ref, tol, "int4")
    assert frac <= 2e-2


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("angle_kind,std", [("uniform", 1.0), ("normal", 0.0)])
def test_tensor_core_composite_5120_angles_and_factors(angle_kind, std, path, monkeypatch):
    _select(monkeypatch, path)
    p, q1, x, y_ref, tol = _tf32_setup(333, seed=9, std=std, angle_kind=angle_kind, path=path)
    y = p.composite_forward(q1, x.to(DEV))
    _check_tf32_rows(y, y_ref, tol, "bf16 rows")
    codes, scales = p.composite_forward_quant(q1, x.to(DEV), 4)
    _check_tf32_quant(codes, scales, y_ref, tol, "int4")
    assert p.device_status() == 0


@pytest.mark.parametrize("path", PATHS)
def test_tensor_core_composite_5120_follows_new_angles_and_the_generic_kernels(path, monkeypatch):
    _select(monkeypatch, path)
    p, q1, x, y_ref, tol = _tf32_setup(200, seed=21, path=path)
    xd = x.to(DEV)
    y1 = p.composite_forward(q1, xd)
    th = synth.angles(128, "uniform", 77)
    p.set_angles(th.to(DEV))
    y2 = p.composite_forward(q1, xd)
    monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
    y2g = p.composite_forward(q1, xd, out_dtype=torch.float32)
    monkeypatch.delenv("BFQ_GENERIC_ONLY")
    assert not torch.equal(y1, y2)
    Q1 = to_f64(q1)
    inner = oracle.forward(to_f64(th), to_f64(x).reshape(-1, 128)).reshape(200, 40, 128)
    tol2 = 2.0 ** -9 * np.einsum("ik,rkj->rij", np.abs(Q1), np.abs(inner)).reshape(200, -1) + 1e-4 * np.abs(to_f64(x)).max()
    _check_tf32_rows(y2, to_f64(y2g), tol2, "tensor-core path against the generic kernels")


@pytest.mark.parametrize("path", PATHS)
def test_tensor_core_composite_5120_padded_rows_and_guards(path, monkeypatch):
    from parity import Guarded
    _select(monkeypatch, path)
    rows = 37
    p, q1, x, y_ref, tol = _tf32_setup(rows, seed=13, path=path)
    xs = torch.zeros((rows, 5120 + 64), dtype=torch.bfloat16, device=DEV)
    xs[:, :5120] = x.to(DEV)
    codes = Guarded((rows, 2560), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    from paper_2509_09679_b200.binding import lib, _check, _stream
    _check(lib().bfq_composite_forward_quant(p._h, q1.data_ptr(), 40, xs.data_ptr(), 1, rows, xs.stride(0), 4,
                                             codes.view.data_ptr(), scales.view.data_ptr(), _stream(xs)), "quant")
    assert p.device_status() == 0
    assert codes.intact() and scales.intact()
    _check_tf32_quant(codes.view, scales.view, y_ref, tol, "int4 with a padded leading dimension")


@pytest.mark.parametrize("path", PATHS)
def test_full_size_composite_5120_sampled(path, monkeypatch):
    """The benchmark's configuration (32768 bf16 token rows of d = 5120, INT4), sampled rows against the oracle."""
    from parity import Guarded
    _select(monkeypatch, path)
    c = synth.COMPOSITE_5120
    n1, n2, rows = c["n1"], c["n2"], c["n_rows"]
    theta2 = synth.angles(n2, "normal", c["seed"], DEV)
    params = synth.cayley_params(n1, c["seed"], device=DEV)
    x = synth.rows(rows, n1 * n2, c["dist"], c["seed"] + 1, outliers=c["outliers"], outlier_scale=c["outlier_scale"],
                   dtype=torch.bfloat16, device=DEV)
    p = Plan(n2, DEV)
    p.set_angles(theta2)
    q1 = p.cayley(params, n1)
    codes = Guarded((rows, 2560), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.composite_forward_quant(q1, x, 4, codes=codes.view, scales=scales.view)
    assert p.device_status() == 0
    assert codes.intact() and scales.intact()
    idx = np.unique(np.concatenate([np.arange(8), np.arange(rows - 8, rows),
                                    np.random.default_rng(0).integers(0, rows, 496)]))
    ti = torch.from_numpy(idx).to(DEV)
    Q1 = oracle.cayley(to_f64(params), n1)
    x64 = to_f64(x[ti])
    inner = oracle.forward(to_f64(theta2), x64.reshape(-1, n2)).reshape(len(idx), n1, n2)
    y_ref = np.einsum("ik,rkj->rij", Q1, inner).reshape(len(idx), -1)
    tol = 2.0 ** -10 * np.einsum("ik,rkj->rij", np.abs(Q1), np.abs(inner)).reshape(len(idx), -1)
    if path == "dense":
        Q2 = oracle.forward(to_f64(theta2), np.eye(n2)).T
        absin = (np.abs(x64).reshape(-1, n2) @ np.abs(Q2).T).reshape(len(idx), n1, n2)
        tol = 2.0 * tol + 2.0 ** -16 * np.einsum("ik,rkj->rij", np.abs(Q1), absin).reshape(len(idx), -1)
    tol = tol + 1e-5 * np.abs(x64).max(axis=1, keepdims=True)
    frac = _check_tf32_quant(codes.view[ti], scales.view[ti], y_ref, tol, "composite 5120 int4, full size")
    assert frac <= 2e-2
    c2, s2 = p.composite_forward_quant(q1, x, 4)  # bit-identical from run to run
    assert torch.equal(c2, codes.view) and torch.equal(s2.view(torch.int16), scales.view.view(torch.int16))


@pytest.mark.parametrize("path", PATHS)
def test_tensor_core_composite_5120_degenerate_rows(path, monkeypatch):
    """Zero rows (scale 0, codes 0), rows so small that the fp16 scale is subnormal, rows so large that it saturates."""
    _select(monkeypatch, path)
    rows = 11
    p, q1, x, _, _ = _tf32_setup(rows, seed=31, path=path)
    xs = x.clone().float()
    xs[1] = 0.0
    xs[2] *= 1e-7
    xs[3] *= 1e-9
    xs[5] *= 1e28
    xs[8] = 0.0
    xs[8, 4097] = 3.0
    x = xs.to(torch.bfloat16)
    x64 = to_f64(x)
    n1, n2 = 40, 128
    th2 = to_f64(synth.angles(n2, "normal", 31))
    Q1 = oracle.cayley(to_f64(synth.cayley_params(n1, 31, 0.1)), n1)
    inner = oracle.forward(th2, x64.reshape(-1, n2)).reshape(rows, n1, n2)
    y_ref = np.einsum("ik,rkj->rij", Q1, inner).reshape(rows, -1)
    tol = 2.0 ** -9 * np.einsum("ik,rkj->rij", np.abs(Q1), np.abs(inner)).reshape(rows, -1)
    Q2 = oracle.forward(th2, np.eye(n2)).T
    absin = (np.abs(x64).reshape(-1, n2) @ np.abs(Q2).T).reshape(rows, n1, n2)
    tol = tol + 2.0 ** -16 * np.einsum("ik,rkj->rij", np.abs(Q1), absin).reshape(rows, -1) + 1e-5 * np.abs(x64).max(axis=1, keepdims=True)
    codes, scales = p.composite_forward_quant(q1, x.to(DEV), 4)
    assert p.device_status() == 0
    s = scales.cpu().view(torch.int16).numpy().view(np.uint16)
    assert s[1] == 0 and not codes[1].any()          # zero row
    assert s[5] == 0x7BFF                              # saturated scale: codes clip
    assert 0 < s[3] < 0x0400 or s[3] == 0              # subnormal (or flushed) scale
    _check_tf32_quant(codes, scales, y_ref, tol, "degenerate rows")
    y = p.composite_forward(q1, x.to(DEV))
    _check_tf32_rows(y, y_ref, tol, "degenerate rows, bf16 out")


# ---- inverse / transpose of the composite ---------------------------------------------------------------------------
@pytest.mark.parametrize("n1,n2,rows", [(3, 16, 7), (12, 256, 33), (40, 128, 61), (7, 1024, 20)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_composite_inverse_generic(n1, n2, rows, dtype, monkeypatch):
    monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
    p, q1, Q1_ref, th2, y = setup(n1, n2, rows, dtype)
    x_ref = oracle.composite_inverse(Q1_ref, th2, to_f64(y))
    amax = np.abs(to_f64(y)).max(axis=1)
    x = p.composite_inverse(q1, y.to(DEV), out_dtype=torch.float32)
    check_rows_close(x, x_ref, amax, "composite inverse")
    # forward(inverse(y)) = y
    back = p.composite_forward(q1, x, out_dtype=torch.float32)
    check_rows_close(back, to_f64(y), np.sqrt(n1 * n2) * amax, "composite round trip")


@pytest.mark.parametrize("rows", [1, 3, 4, 593, 2500])
def test_tensor_core_composite_inverse_5120(rows):
    n1, n2 = 40, 128
    p, q1, y, _, _ = _tf32_setup(rows, seed=41, path="dense")
    th2 = to_f64(synth.angles(n2, "normal", 41))
    Q1 = oracle.cayley(to_f64(synth.cayley_params(n1, 41, 0.1)), n1)
    y64 = to_f64(y)
    x_ref = oracle.composite_inverse(Q1, th2, y64)
    # same error model as the forward dense path, with the transposed factors
    inner = oracle.inverse(th2, y64.reshape(-1, n2)).reshape(rows, n1, n2)
    Q2 = oracle.forward(th2, np.eye(n2)).T
    absin = (np.abs(y64).reshape(-1, n2) @ np.abs(Q2)).reshape(rows, n1, n2)
    tol = 2.0 ** -9 * np.einsum("ki,rkj->rij", np.abs(Q1), np.abs(inner)).reshape(rows, -1) \
        + 2.0 ** -16 * np.einsum("ki,rkj->rij", np.abs(Q1), absin).reshape(rows, -1) + 1e-5 * np.abs(y64).max(axis=1, keepdims=True)
    x = p.composite_inverse(q1, y.to(DEV))
    assert p.device_status() == 0
    _check_tf32_rows(x, x_ref, tol, "tensor-core composite inverse")
    # adjoint identity <Q x, z> = <x, Q^T z> on the device results, in float64, within the two paths' tolerances
    z = p.composite_forward(q1, y.to(DEV))
    lhs = (to_f64(z) * y64).sum(axis=1)
    rhs = (y64 * to_f64(x)).sum(axis=1)
    assert np.all(np.abs(lhs - rhs) <= 2e-2 * (np.abs(y64) ** 2).sum(axis=1))


# ---- gradients of the composite, composed from the entry points --------------------------------------------------------
def test_composite_backward_against_float64_and_finite_differences():
    from paper_2509_09679_b200.composite import cayley_pullback, composite_backward
    n1, n2, tokens = 6, 64, 37
    theta2 = synth.angles(n2, "normal", 3)
    params = synth.cayley_params(n1, 3, 0.3)
    x = synth.rows(tokens, n1 * n2, "normal", 4)
    g = synth.rows(tokens, n1 * n2, "normal", 5)
    p = Plan(n2, DEV)
    p.set_angles(theta2.to(DEV))
    q1 = p.cayley(params.to(DEV), n1)
    dx, dth2, dQ1, dpar = composite_backward(p, q1, params.to(DEV), x.to(DEV), g.to(DEV))
    # float64 reference from the oracle's pieces: L(theta2, params) = sum(g * composite_forward(x))
    th64, x64, g64, par64 = to_f64(theta2), to_f64(x), to_f64(g), to_f64(params)
    Q1 = oracle.cayley(par64, n1)
    check_rows_close(dx, oracle.composite_inverse(Q1, th64, g64), np.abs(g64).max(axis=1), "composite dx")
    gp = np.einsum("ki,rkj->rij", Q1, g64.reshape(tokens, n1, n2)).reshape(-1, n2)
    _, dth_ref = oracle.backward(th64, x64.reshape(-1, n2), gp)
    from parity import check_dtheta
    check_dtheta(dth2, dth_ref, "composite dtheta2")
    xp = oracle.forward(th64, x64.reshape(-1, n2)).reshape(tokens, n1, n2)
    dQ1_ref = np.einsum("rij,rkj->ik", g64.reshape(tokens, n1, n2), xp)
    assert np.abs(to_f64(dQ1) - dQ1_ref).max() <= 1e-4 * np.abs(dQ1_ref).max()
    # the Cayley pull-back against central differences of the oracle (CPU, float64)
    loss = lambda q: float(np.sum(g64 * oracle.composite_forward(oracle.cayley(q, n1), th64, x64)))
    fd = np.zeros_like(par64)
    for k in range(par64.size):
        e = np.zeros_like(par64)
        e[k] = 1e-6
        fd[k] = (loss(par64 + e) - loss(par64 - e)) / 2e-6
    got = to_f64(cayley_pullback(torch.from_numpy(par64), n1, torch.from_numpy(dQ1_ref)))
    assert np.abs(got - fd).max() <= 1e-6 * max(1.0, np.abs(fd).max())
    assert np.abs(to_f64(dpar) - fd).max() <= 2e-4 * np.abs(fd).max()


@pytest.mark.parametrize("rows", [1, 3, 5, 593, 2500])
def test_tensor_core_composite_5120_int8(rows):
    p, q1, x, y_ref, tol = _tf32_setup(rows, seed=17, path="dense")
    if rows >= 5:
        xs = x.float()
        xs[1] = 0.0
        xs[2] *= 1e-9
        xs[3] *= 1e28
        x = xs.to(torch.bfloat16)
        p, q1, _, _, _ = _tf32_setup(rows, seed=17, path="dense")
        x64 = to_f64(x)
        th2 = to_f64(synth.angles(128, "normal", 17))
        Q1 = oracle.cayley(to_f64(synth.cayley_params(40, 17, 0.1)), 40)
        inner = oracle.forward(th2, x64.reshape(-1, 128)).reshape(rows, 40, 128)
        y_ref = np.einsum("ik,rkj->rij", Q1, inner).reshape(rows, -1)
        Q2 = oracle.forward(th2, np.eye(128)).T
        absin = (np.abs(x64).reshape(-1, 128) @ np.abs(Q2).T).reshape(rows, 40, 128)
        tol = 2.0 ** -9 * np.einsum("ik,rkj->rij", np.abs(Q1), np.abs(inner)).reshape(rows, -1) \
            + 2.0 ** -16 * np.einsum("ik,rkj->rij", np.abs(Q1), absin).reshape(rows, -1) + 1e-5 * np.abs(x64).max(axis=1, keepdims=True)
    from parity import Guarded
    codes = Guarded((rows, 5120), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    from paper_2509_09679_b200.binding import lib, _check, _stream
    xd = x.to(DEV)
    _check(lib().bfq_composite_forward_quant(p._h, q1.data_ptr(), 40, xd.data_ptr(), 1, rows, 5120, 8, codes.view.data_ptr(),
                                             scales.view.data_ptr(), _stream(xd)), "int8")
    assert p.device_status() == 0 and codes.intact() and scales.intact()
    frac = _check_tf32_quant(codes.view, scales.view, y_ref, tol, "composite int8", bits=8)
    assert frac <= 0.2  # codes are 16 times finer than INT4: the TF32 error moves proportionally more of them by one
