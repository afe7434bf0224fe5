"""GPU parity, second part: the two rotation forms of the tuned kernels (scaled two-FMA form and the three-shear
fallback), the stated checks of the full-size configurations, the tuned-versus-generic cross-check, and the bounded
device wait.  Rules are in parity.py."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2509_09679_b200 import Plan, synth
from parity import Guarded, check_dtheta, check_quant, check_rows_close, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def absmax_rows(x):
    return np.abs(to_f64(x)).max(axis=1)


def angle_set(kind, n, seed):
    """Angle sets chosen by how the scaled form treats them (n log2 n / 2 angles, Sec. 3.2.1)."""
    L = n.bit_length() - 1
    g = torch.Generator().manual_seed(seed)
    if kind == "small":        # every |theta| <= pi/4: every multiplier |tan| <= 1, factors >= 2^-(L/2)
        return (torch.rand((L, n // 2), generator=g) * 2 - 1) * (math.pi / 4)
    if kind == "steep":        # |theta| = pi/2 - 0.03: |tan| = 33 in every pair, factors down to 0.03^11
        sign = torch.randint(0, 2, (L, n // 2), generator=g) * 2 - 1
        return sign * (math.pi / 2 - 0.03)
    if kind == "singular":     # |theta| = pi/2 - 1e-4 everywhere: the factors leave 2^-64 -> three-shear fallback
        sign = torch.randint(0, 2, (L, n // 2), generator=g) * 2 - 1
        return sign * (math.pi / 2 - 1e-4)
    if kind == "hadamard":     # all pi/4 (the Hadamard special case of the paper's theorem): factor 2^-(L/2)
        return torch.full((L, n // 2), math.pi / 4)
    if kind == "uniform":      # U[-pi, pi): large dynamic range of factors, still in range with overwhelming odds
        return (torch.rand((L, n // 2), generator=g) * 2 - 1) * math.pi
    raise ValueError(kind)


# expected bfq_stage_form bit 0 (forward tables) per angle set
FORWARD_FALLBACK = {"small": 0, "steep": 0, "singular": 1, "hadamard": 0, "uniform": 0}


@pytest.mark.parametrize("kind", ["small", "steep", "singular", "hadamard", "uniform"])
def test_rotation_forms_n4096(kind):
    n, rows = 4096, 301
    theta = angle_set(kind, n, 700).float()
    x = synth.rows(rows, n, "student_t3", 701, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    th64, x64 = to_f64(theta), to_f64(x)
    p = Plan(n, DEV)
    p.set_angles(theta.to(DEV))
    xd = x.to(DEV)
    y_ref = oracle.forward(th64, x64)
    codes, scales = p.forward_quant(xd, 4)
    check_quant(codes, scales, y_ref, 4, f"{kind} INT4")
    codes2, scales2 = p.forward_quant(xd, 2)
    check_quant(codes2, scales2, y_ref, 2, f"{kind} INT2")
    check_rows_close(p.forward(xd), y_ref, absmax_rows(x), f"{kind} bf16 rows")
    # inverse / transpose (its own tables and range flag)
    check_rows_close(p.inverse(xd, out_dtype=torch.float32), oracle.inverse(th64, x64), absmax_rows(x), f"{kind} inverse")
    form = p.stage_form()
    assert (form & 1) == FORWARD_FALLBACK[kind], f"{kind}: forward form {form}"
    assert ((form >> 1) & 1) == FORWARD_FALLBACK[kind], f"{kind}: inverse form {form}"
    assert p.device_status() == 0


@pytest.mark.parametrize("kind", ["small", "steep", "singular", "uniform"])
def test_rotation_forms_n8192(kind):
    n, rows = 8192, 151
    theta = angle_set(kind, n, 710).float()
    x = synth.rows(rows, n, "laplace", 711, outliers=16, outlier_scale=100.0, dtype=torch.bfloat16)
    p = Plan(n, DEV)
    p.set_angles(theta.to(DEV))
    y_ref = oracle.forward(to_f64(theta), to_f64(x))
    for bits in (2, 4):
        codes, scales = p.forward_quant(x.to(DEV), bits)
        check_quant(codes, scales, y_ref, bits, f"{kind} n=8192 INT{bits}")
    check_rows_close(p.forward(x.to(DEV)), y_ref, absmax_rows(x), f"{kind} n=8192 bf16 rows")
    # twelve scaled stages per half (the thirteenth is a general 2x2): 0.03^12 = 2^-60.7 is still in range
    assert (p.stage_form() & 1) == (1 if kind == "singular" else 0)
    assert p.device_status() == 0


def test_form_follows_new_angles():
    """The flag is rebuilt by every bfq_set_angles: fallback -> scaled -> fallback on one plan."""
    n = 4096
    x = synth.rows(64, n, "normal", 721, dtype=torch.bfloat16)
    p = Plan(n, DEV)
    for kind, expect in (("singular", 1), ("small", 0), ("singular", 1), ("uniform", 0)):
        theta = angle_set(kind, n, 722).float()
        p.set_angles(theta.to(DEV))
        codes, scales = p.forward_quant(x.to(DEV), 4)
        check_quant(codes, scales, oracle.forward(to_f64(theta), to_f64(x)), 4, f"sequence {kind}")
        assert (p.stage_form() & 1) == expect


def test_tuned_and_generic_kernels_agree_int4_n4096(monkeypatch):
    """The tuned n = 4096 INT4 path against the generic kernel of the same library on the headline rows: equal scales
    except where the fp32 absmax lands either side of an fp16 rounding boundary, codes different in < 1e-3 of elements."""
    wl = synth.WORKLOADS["act4096_int4"]
    rows = 8192
    theta = wl.theta(device=DEV)
    x = wl.x(device=DEV, n_rows=rows)
    p = Plan(wl.n, DEV)
    p.set_angles(theta)
    c_t, s_t = p.forward_quant(x, 4)
    monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
    c_g, s_g = p.forward_quant(x, 4)
    monkeypatch.delenv("BFQ_GENERIC_ONLY")
    torch.cuda.synchronize()
    ds = (s_t.view(torch.int16).int() - s_g.view(torch.int16).int()).abs()
    assert int(ds.max()) <= 1 and int((ds != 0).sum()) <= rows // 100
    same_scale = ds == 0
    a = torch.from_numpy(oracle.unpack(c_t[same_scale].cpu().numpy(), 4).astype(np.int16))
    b = torch.from_numpy(oracle.unpack(c_g[same_scale].cpu().numpy(), 4).astype(np.int16))
    d = (a - b).abs()
    assert int(d.max()) <= 1 and float((d != 0).float().mean()) < 1e-3
    assert p.device_status() == 0


def test_fold8192_int2_invariance_check_full_size():
    """Weight folding as the workload states it: W (28672 x 8192 bf16, N(0, 0.02^2)) -> W Q^T -> per-row INT2, checked by
    dequant(W Q^T) (Q x) against W x on 256 vectors x (computational invariance, Sec. 3.1).  INT2 round-to-nearest is
    coarse by construction, so the pass criterion is the oracle's own error level on the same rows, plus the
    unquantized product within bf16 rounding."""
    wl = synth.WORKLOADS["fold8192_int2"]
    theta = wl.theta(device=DEV)
    W = wl.x(device=DEV)
    p = Plan(wl.n, DEV)
    p.set_angles(theta)
    codes, scales, _ = p.fold_weights(W, 2)                      # tuned kernel, the timed configuration
    th64 = to_f64(theta)
    # 256 check vectors: half with the n = 8192 activation distribution, half N(0, 1)
    xa = synth.rows(128, wl.n, "laplace", 5301, outliers=16, outlier_scale=100.0, dtype=torch.bfloat16)
    xb = synth.rows(128, wl.n, "normal", 5302, dtype=torch.bfloat16)
    x = torch.cat([xa, xb]).to(DEV)
    Qx = p.forward(x, out_dtype=torch.float32)                   # fp32 rows: the generic kernel
    Qx_ref = oracle.forward(th64, to_f64(x))
    check_rows_close(Qx, Qx_ref, absmax_rows(x), "Q x")
    # oracle side on a fixed sample of 1024 weight rows
    idx = np.unique(np.concatenate([np.arange(0, wl.n_rows, wl.n_rows // 1008), np.arange(8), np.arange(wl.n_rows - 8, wl.n_rows)]))
    ti = torch.from_numpy(idx).to(DEV)
    W64 = to_f64(W[ti])
    WQt_ref = oracle.forward(th64, W64)
    check_quant(codes[ti], scales[ti], WQt_ref, 2, "fold8192 codes")
    ref = W64 @ to_f64(x).T                                       # W x, [sample][256]
    o_codes, o_scales = oracle.quantize(WQt_ref, 2)
    err_ref = np.linalg.norm(oracle.dequantize(o_codes, o_scales) @ Qx_ref.T - ref) / np.linalg.norm(ref)
    deq = oracle.dequantize(oracle.unpack(codes[ti].cpu().numpy(), 2),
                            scales[ti].cpu().view(torch.int16).numpy().view(np.uint16))
    err_gpu = np.linalg.norm(deq @ to_f64(Qx).T - ref) / np.linalg.norm(ref)
    assert abs(err_gpu - err_ref) <= 1e-3 * err_ref, (err_gpu, err_ref)
    assert p.device_status() == 0
    # unquantized leg: bf16 W Q^T (rotated rows kept) times Q x against W x, within bf16 rounding of the rows
    _, _, rot = p.fold_weights(W[ti], 2, want_rotated=True)
    check_rows_close(rot, WQt_ref, absmax_rows(W[ti]), "W Q^T bf16")
    prod = to_f64(rot) @ to_f64(Qx).T
    scale = np.sqrt((W64 ** 2).sum(axis=1, keepdims=True)) * np.sqrt((to_f64(x) ** 2).sum(axis=1))[None, :]
    assert np.abs(prod - ref).max() <= 2.0 ** -8 * scale.max(), "unquantized (W Q^T)(Q x) vs W x"


@pytest.mark.slow
def test_learn4096_backward_all_rows():
    """The angle-learning step on all 128 x 2048 rows: d-theta reduced over every row against the oracle summed over
    32 row blocks; dL/dx on sampled rows."""
    wl = synth.WORKLOADS["learn4096"]
    theta = wl.theta(device=DEV)
    x = wl.x(device=DEV)
    g = wl.g(device=DEV)
    p = Plan(wl.n, DEV)
    p.set_angles(theta)
    dx = torch.empty_like(x)
    dth = Guarded((wl.L, wl.n // 2), torch.float32, DEV)
    p.backward(x, g, dx=dx, dtheta=dth.view)
    assert p.device_status() == 0 and dth.intact()
    th64 = to_f64(theta)
    acc = np.zeros((wl.L, wl.n // 2))
    for r0 in range(0, wl.n_rows, 8192):
        acc += oracle.backward(th64, to_f64(x[r0:r0 + 8192]), to_f64(g[r0:r0 + 8192]))[1]
    check_dtheta(dth.view, acc, "learn4096 dtheta, all rows")
    idx = np.arange(0, wl.n_rows, wl.n_rows // 512)
    ti = torch.from_numpy(idx).to(DEV)
    dx_ref, _ = oracle.backward(th64, to_f64(x[ti]), to_f64(g[ti]))
    check_rows_close(dx[ti], dx_ref, absmax_rows(g[ti]), "learn4096 dx")


@pytest.mark.slow
def test_act8192_backward_and_inverse_at_the_timed_sizes():
    """The two n = 8192 legs the benchmark times, in its launch configuration: backward on a quarter of the activation
    rows (d-theta over every row against the oracle summed over row blocks, dL/dx on sampled rows), inverse on all of
    them (sampled rows)."""
    wl = synth.WORKLOADS["act8192_int2"]
    theta = wl.theta(device=DEV)
    x = wl.x(device=DEV)
    p = Plan(wl.n, DEV)
    p.set_angles(theta)
    th64 = to_f64(theta)
    rows = wl.n_rows // 4
    g = wl.g(device=DEV, n_rows=rows)
    dx = torch.empty_like(g)
    dth = Guarded((wl.L, wl.n // 2), torch.float32, DEV)
    p.backward(x[:rows], g, dx=dx, dtheta=dth.view)
    assert p.device_status() == 0 and dth.intact()
    acc = np.zeros((wl.L, wl.n // 2))
    for r0 in range(0, rows, 2048):
        acc += oracle.backward(th64, to_f64(x[r0:r0 + 2048]), to_f64(g[r0:r0 + 2048]))[1]
    check_dtheta(dth.view, acc, "act8192 dtheta, all rows of the timed batch")
    ti = torch.from_numpy(np.arange(0, rows, rows // 256)).to(DEV)
    dx_ref, _ = oracle.backward(th64, to_f64(x[ti]), to_f64(g[ti]))
    check_rows_close(dx[ti], dx_ref, absmax_rows(g[ti]), "act8192 dx")
    del g, dx
    out = torch.empty_like(x)
    p.inverse(x, out=out)
    assert p.device_status() == 0
    ti = torch.from_numpy(np.arange(0, wl.n_rows, wl.n_rows // 256)).to(DEV)
    check_rows_close(out[ti], oracle.inverse(th64, to_f64(x[ti])), absmax_rows(x[ti]), "act8192 inverse")
    ti = torch.tensor([0, 1, 2, 3, wl.n_rows - 4, wl.n_rows - 3, wl.n_rows - 2, wl.n_rows - 1], device=DEV)  # first and last CTA
    check_rows_close(out[ti], oracle.inverse(th64, to_f64(x[ti])), absmax_rows(x[ti]), "act8192 inverse, ends")


def test_bounded_wait_runs_out_and_the_plan_recovers():
    """A device-side wait that cannot be satisfied (the kernel is told to expect 16 bytes more per row load than
    arrive) gives up after its poll limit: the kernel returns, the status word reports it once, nothing is written
    outside the outputs, and the next ordinary call on the same plan is correct.  No trap, no unbounded spin."""
    n, rows = 4096, 4
    theta = synth.angles(n, "normal", 731)
    x = synth.rows(rows, n, "student_t3", 732, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    p = Plan(n, DEV)
    p.set_angles(theta.to(DEV))
    codes = Guarded((rows, n // 2), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.test_stuck_wait(True)
    p.forward_quant(x.to(DEV), 4, codes=codes.view, scales=scales.view)
    torch.cuda.synchronize()                       # the kernel returned
    assert p.device_status() == -9                 # BFQ_ERR_DEVICE_TIMEOUT, reported once ...
    assert p.device_status() == 0                  # ... and cleared
    assert codes.intact() and scales.intact()
    p.test_stuck_wait(False)
    p.forward_quant(x.to(DEV), 4, codes=codes.view, scales=scales.view)
    check_quant(codes.view, scales.view, oracle.forward(to_f64(theta), to_f64(x)), 4, "after a timed-out call")
    assert p.device_status() == 0 and codes.intact() and scales.intact()
