"""GPU parity: every entry point of the C ABI against the CPU oracle, element by element,
on seeded inputs.  Sizes span several tiles and ragged tails; the rules are in parity.py."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_09679_b200 import BfqError, Plan, synth
from parity import Guarded, check_dtheta, check_quant, check_rows_close, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make(n, rows, dtype, dist="student_t3", angle_kind="normal", seed=1, outliers=4, oscale=20.0):
    theta = synth.angles(n, angle_kind, seed)
    x = synth.rows(rows, n, dist, seed + 1, outliers=min(outliers, n // 4), outlier_scale=oscale, dtype=dtype)
    return theta, x


def plan_for(n, theta):
    p = Plan(n, DEV)
    p.set_angles(theta.to(DEV))
    return p


def absmax_rows(x):
    return np.abs(to_f64(x)).max(axis=1) if x.shape[0] else np.zeros(0)


# ---- the tiny correctness configuration: n = 256, 1024 fp32 rows, angles U[-pi, pi) ------------------
def test_tiny256_all_entry_points():
    wl = synth.WORKLOADS["tiny256"]
    theta, x, g = wl.theta(), wl.x(), wl.g()
    th64, x64, g64 = to_f64(theta), to_f64(x), to_f64(g)
    p = plan_for(wl.n, theta)
    xd, gd = x.to(DEV), g.to(DEV)
    y_ref = oracle.forward(th64, x64)
    y = p.forward(xd)
    check_rows_close(y, y_ref, absmax_rows(x), "forward")
    xr = p.inverse(y)
    check_rows_close(xr, oracle.inverse(th64, to_f64(y)), absmax_rows(y), "inverse")
    check_rows_close(xr, x64, np.sqrt(wl.n) * absmax_rows(x), "round trip")
    codes, scales = p.forward_quant(xd, 4)
    stats = check_quant(codes, scales, y_ref, 4, "forward_quant")
    assert stats["scale_ulp_rows"] <= 16
    dx, dth = p.backward(xd, gd)
    dx_ref, dth_ref = oracle.backward(th64, x64, g64)
    check_rows_close(dx, dx_ref, absmax_rows(g), "dx")
    check_dtheta(dth, dth_ref, "dtheta")
    assert p.device_status() == 0


# ---- every supported n, both dtypes, ragged row counts, padded leading dimension ----------------------
@pytest.mark.parametrize("n", [16, 32, 64, 128, 256, 512, 1024, 2048, 4096, 8192])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_forward_inverse_every_n(n, dtype):
    rows = 67 if n >= 2048 else 333
    theta, x = make(n, rows, dtype, angle_kind="uniform", seed=n)
    th64 = to_f64(theta)
    p = plan_for(n, theta)
    ld = n + 24
    xpad = torch.zeros((rows, ld), dtype=dtype, device=DEV)
    xpad[:, :n] = x.to(DEV)
    xv = xpad[:, :n]
    y_ref = oracle.forward(th64, to_f64(x))
    for out_dtype in (torch.float32, torch.bfloat16):
        out = Guarded((rows, n), out_dtype, DEV)
        p.forward(xv, out=out.view)
        check_rows_close(out.view, y_ref, absmax_rows(x), f"forward n={n} {dtype}->{out_dtype}")
        assert out.intact()
    xi_ref = oracle.inverse(th64, to_f64(x))
    out = Guarded((rows, n), torch.float32, DEV)
    p.inverse(xv, out=out.view)
    check_rows_close(out.view, xi_ref, absmax_rows(x), f"inverse n={n}")
    assert out.intact()
    assert p.device_status() == 0


@pytest.mark.parametrize("n,rows", [(16, 5), (64, 1), (128, 1000), (256, 129), (1024, 77), (4096, 130), (8192, 35)])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_forward_quant_every_width(n, rows, bits):
    theta, x = make(n, rows, torch.bfloat16, seed=7 * n + bits)
    p = plan_for(n, theta)
    y_ref = oracle.forward(to_f64(theta), to_f64(x))
    codes = Guarded((rows, n * bits // 8), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.forward_quant(x.to(DEV), bits, codes=codes.view, scales=scales.view)
    check_quant(codes.view, scales.view, y_ref, bits, f"n={n} bits={bits}")
    assert codes.intact() and scales.intact()


@pytest.mark.parametrize("n,rows", [(16, 9), (128, 300), (512, 70), (2048, 45), (4096, 40), (8192, 20)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_backward_every_n(n, rows, dtype):
    theta, x = make(n, rows, dtype, angle_kind="uniform", seed=3 * n)
    g = synth.rows(rows, n, "normal", 99 + n, dtype=dtype)
    p = plan_for(n, theta)
    dx_ref, dth_ref = oracle.backward(to_f64(theta), to_f64(x), to_f64(g))
    dx = Guarded((rows, n), dtype, DEV)
    dth = Guarded((p.L, n // 2), torch.float32, DEV)
    p.backward(x.to(DEV), g.to(DEV), dx=dx.view, dtheta=dth.view)
    check_rows_close(dx.view, dx_ref, absmax_rows(g), f"dx n={n}")
    check_dtheta(dth.view, dth_ref, f"dtheta n={n}")
    assert dx.intact() and dth.intact()
    # dtheta only
    _, dth2 = p.backward(x.to(DEV), g.to(DEV), want_dx=False)
    assert torch.equal(dth2, dth.view)


def test_backward_is_bit_reproducible():
    n, rows = 4096, 3000
    theta, x = make(n, rows, torch.bfloat16, seed=5)
    g = synth.rows(rows, n, "normal", 6, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    xd, gd = x.to(DEV), g.to(DEV)
    dx1, d1 = p.backward(xd, gd)
    dx2, d2 = p.backward(xd, gd)
    assert torch.equal(d1, d2) and torch.equal(dx1.view(torch.int16), dx2.view(torch.int16))
    assert p.backward_partials() > 0


# ---- special angle sets ---------------------------------------------------------------------------------
@pytest.mark.parametrize("n", [256, 4096])
def test_identity_and_hadamard_angles(n):
    x = synth.rows(50, n, "normal", 3, dtype=torch.float32)
    p = plan_for(n, synth.angles(n, "zero", 0))
    assert torch.equal(p.forward(x.to(DEV)).cpu(), x)  # theta = 0: exact identity
    p.set_angles(synth.angles(n, "hadamard", 0).to(DEV))
    eye = torch.zeros((64, n), dtype=torch.float32)
    eye[torch.arange(64), torch.arange(64) * (n // 64)] = 1.0
    y = p.forward(eye.to(DEV)).cpu()
    assert torch.allclose(y.abs(), torch.full_like(y, 1 / math.sqrt(n)), rtol=0, atol=1e-6)  # coherence 1/sqrt(n)
    np.testing.assert_allclose(np.linalg.norm(to_f64(p.forward(x.to(DEV))), axis=1),
                               np.linalg.norm(to_f64(x), axis=1), rtol=1e-5)


# ---- degenerate rows ---------------------------------------------------------------------------------------
def test_zero_rows_tiny_rows_and_saturating_rows():
    n = 512
    theta, x = make(n, 8, torch.float32, seed=11)
    x[0] = 0.0
    x[1] = x[1] * 1e-12   # scale underflows fp16: codes must be all zero
    x[2] = x[2] * 1e5     # amax/qmax above 65504 for INT2: scale saturates, codes clip
    x[3] = x[3] * 1e-6    # subnormal fp16 scale
    p = plan_for(n, theta)
    y_ref = oracle.forward(to_f64(theta), to_f64(x))
    for bits in (2, 4, 8):
        codes, scales = p.forward_quant(x.to(DEV), bits)
        check_quant(codes, scales, y_ref, bits, f"degenerate bits={bits}")
        assert not codes[0].any() and scales[0].item() == 0


def test_zero_row_count_and_single_row():
    n = 1024
    theta, x = make(n, 1, torch.bfloat16, seed=12)
    p = plan_for(n, theta)
    empty = torch.empty((0, n), dtype=torch.bfloat16, device=DEV)
    assert p.forward(empty).shape == (0, n)
    c, s = p.forward_quant(empty, 4)
    assert c.shape == (0, n // 2) and s.shape == (0,)
    dx, dth = p.backward(empty, empty)
    assert not dth.any()
    y = p.forward(x.to(DEV), out_dtype=torch.float32)
    check_rows_close(y, oracle.forward(to_f64(theta), to_f64(x)), absmax_rows(x), "single row")


# ---- argument validation (host side, before any launch) ----------------------------------------------------
def test_argument_validation_codes():
    n = 256
    theta, x = make(n, 4, torch.float32)
    with pytest.raises(BfqError) as e:
        Plan(100, DEV)
    assert e.value.status == -2
    p = Plan(n, DEV)
    xd = x.to(DEV)
    with pytest.raises(BfqError) as e:  # angles not set
        p.forward(xd)
    assert e.value.status == -7
    p.set_angles(theta.to(DEV))
    with pytest.raises(BfqError) as e:
        p.forward_quant(xd, 3)
    assert e.value.status == -3
    mis = torch.empty(4 * n + 1, dtype=torch.float32, device=DEV)[1:].view(4, n)
    with pytest.raises(BfqError) as e:
        p.forward(mis)
    assert e.value.status == -4
    with pytest.raises(TypeError):
        p.forward(xd.to(torch.float16))
    bad_ld = torch.empty((4, n + 1), dtype=torch.float32, device=DEV)[:, :n]
    with pytest.raises(BfqError) as e:
        p.forward(bad_ld)
    assert e.value.status == -5
    assert p.device_status() == 0


# ---- weight folding: (W Q^T)(Q x) = W x ---------------------------------------------------------------------
def test_fold_weights_small():
    n, m = 1024, 96
    theta = synth.angles(n, "normal", 21)
    W = synth.rows(m, n, "normal", 22, scale=0.02, dtype=torch.bfloat16)
    x = synth.rows(32, n, "laplace", 23, outliers=4, outlier_scale=100.0, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    th64 = to_f64(theta)
    codes, scales, rot = p.fold_weights(W.to(DEV), 2, want_rotated=True, rotated_dtype=torch.float32)
    WQt_ref = oracle.forward(th64, to_f64(W))
    check_rows_close(rot, WQt_ref, absmax_rows(W), "W Q^T")
    check_quant(codes, scales, WQt_ref, 2, "fold codes")
    Qx = to_f64(p.forward(x.to(DEV), out_dtype=torch.float32))
    ref = to_f64(W) @ to_f64(x).T
    np.testing.assert_allclose(to_f64(rot) @ Qx.T, ref, atol=1e-4 * np.abs(ref).max())
    # quantized product: same error level as the oracle's own quantized product
    o_codes, o_scales = oracle.quantize(WQt_ref, 2)
    err_ref = np.linalg.norm(oracle.dequantize(o_codes, o_scales) @ oracle.forward(th64, to_f64(x)).T - ref)
    deq = oracle.dequantize(oracle.unpack(codes.cpu().numpy(), 2), scales.cpu().view(torch.int16).numpy().view(np.uint16))
    err_gpu = np.linalg.norm(deq @ Qx.T - ref)
    assert abs(err_gpu - err_ref) <= 1e-3 * err_ref


# ---- full-size workloads, in the launch configuration the benchmark times --------------------------------
def _sample_rows(n_rows, count):
    idx = np.unique(np.concatenate([np.arange(0, n_rows, max(1, n_rows // count)), np.arange(min(n_rows, 8)),
                                    np.arange(max(0, n_rows - 8), n_rows)]))
    return idx


def test_full_size_forward_int4_n4096():
    wl = synth.WORKLOADS["act4096_int4"]
    theta = wl.theta(device=DEV)
    x = wl.x(device=DEV)
    p = Plan(wl.n, DEV)
    p.set_angles(theta)
    codes = Guarded((wl.n_rows, wl.n // 2), torch.uint8, DEV)
    scales = Guarded((wl.n_rows,), torch.float16, DEV)
    p.forward_quant(x, 4, codes=codes.view, scales=scales.view)
    assert p.device_status() == 0
    assert codes.intact() and scales.intact()
    idx = _sample_rows(wl.n_rows, 4096)
    ti = torch.from_numpy(idx).to(DEV)
    y_ref = oracle.forward(to_f64(theta), to_f64(x[ti]))
    stats = check_quant(codes.view[ti], scales.view[ti], y_ref, 4, "act4096_int4")
    assert stats["scale_ulp_rows"] <= max(4, len(idx) // 100)
    # run twice: identical bits
    c2, s2 = p.forward_quant(x, 4)
    assert torch.equal(c2, codes.view) and torch.equal(s2.view(torch.int16), scales.view.view(torch.int16))
    # the tuned path and the generic path must agree on the scales (same fp32 absmax up to rounding order)
    ds = (s2.view(torch.int16).int() - scales.view.view(torch.int16).int()).abs().max().item()
    assert ds == 0


@pytest.mark.parametrize("rows", [1, 2, 3, 5, 147, 148 * 3 + 1, 1000])
@pytest.mark.parametrize("angle_kind", ["normal", "uniform"])
def test_tuned_n4096_ragged_row_counts(rows, angle_kind):
    n = 4096
    theta = synth.angles(n, angle_kind, 40 + rows)
    x = synth.rows(rows, n, "student_t3", 41 + rows, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    ld = n + 8
    xpad = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    xpad[:, :n] = x.to(DEV)
    codes = Guarded((rows, n // 2), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.forward_quant(xpad[:, :n], 4, codes=codes.view, scales=scales.view)
    assert p.device_status() == 0
    check_quant(codes.view, scales.view, oracle.forward(to_f64(theta), to_f64(x)), 4, f"tuned rows={rows}")
    assert codes.intact() and scales.intact()


def test_tuned_n4096_special_angles_and_degenerate_rows():
    n = 4096
    x = synth.rows(64, n, "normal", 77, dtype=torch.bfloat16)
    x[0] = 0
    x[1] *= 1e-9
    x[2] *= 1e6
    x[3] *= 3e-5
    for kind, seed in (("zero", 0), ("hadamard", 0), ("uniform", 5)):
        theta = synth.angles(n, kind, seed)
        if kind == "uniform":  # exact multiples of pi/2 and pi exercise the angle reduction
            theta[:, ::7] = math.pi / 2
            theta[:, 1::7] = -math.pi
            theta[:, 2::7] = math.pi
            theta[:, 3::7] = -math.pi / 2
            theta[:, 4::7] = 100.0
        p = plan_for(n, theta)
        codes, scales = p.forward_quant(x.to(DEV), 4)
        check_quant(codes, scales, oracle.forward(to_f64(theta), to_f64(x)), 4, f"tuned {kind}")
        assert p.device_status() == 0


# ---- tuned backward for n = 4096 bf16 rows ------------------------------------------------------------------
@pytest.mark.parametrize("rows", [1, 2, 3, 295, 296, 297, 1001])
@pytest.mark.parametrize("angle_kind", ["normal", "uniform"])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_tuned_backward_n4096_ragged_row_counts(rows, angle_kind, dtype):
    n = 4096
    theta = synth.angles(n, angle_kind, 60 + rows)
    if angle_kind == "uniform":  # exact multiples of pi/2 and pi exercise the angle reduction and its sign tracking
        theta[:, ::7] = math.pi / 2
        theta[:, 1::7] = -math.pi
        theta[:, 2::7] = math.pi
        theta[:, 3::7] = -math.pi / 2
        theta[:, 4::7] = 100.0
    x = synth.rows(rows, n, "student_t3", 61 + rows, outliers=8, outlier_scale=50.0, dtype=dtype)
    g = synth.rows(rows, n, "normal", 62 + rows, dtype=dtype)
    p = plan_for(n, theta)
    ld = n + 8
    xpad = torch.zeros((rows, ld), dtype=dtype, device=DEV)
    gpad = torch.zeros((rows, ld), dtype=dtype, device=DEV)
    xpad[:, :n] = x.to(DEV)
    gpad[:, :n] = g.to(DEV)
    dxbuf = Guarded((rows, ld), dtype, DEV)
    dth = Guarded((p.L, n // 2), torch.float32, DEV)
    p.backward(xpad[:, :n], gpad[:, :n], dx=dxbuf.view[:, :n], dtheta=dth.view)
    assert p.device_status() == 0
    dx_ref, dth_ref = oracle.backward(to_f64(theta), to_f64(x), to_f64(g))
    check_rows_close(dxbuf.view[:, :n], dx_ref, absmax_rows(g), f"tuned dx rows={rows}")
    check_dtheta(dth.view, dth_ref, f"tuned dtheta rows={rows}")
    assert dxbuf.intact() and dth.intact()
    assert (dxbuf.view[:, n:].contiguous().view(torch.int16) == torch.tensor(0xA5A5, dtype=torch.uint16).view(torch.int16)).all()
    assert p.backward_partials() == min((rows + 1) // 2, torch.cuda.get_device_properties(0).multi_processor_count)
    # d-theta only, and again: same bits
    _, dth2 = p.backward(xpad[:, :n], gpad[:, :n], want_dx=False)
    assert torch.equal(dth2, dth.view)


def test_tuned_backward_follows_new_angles_and_agrees_with_the_generic_kernels(monkeypatch):
    n, rows = 4096, 500
    x = synth.rows(rows, n, "student_t3", 71, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16).to(DEV)
    g = synth.rows(rows, n, "normal", 72, dtype=torch.bfloat16).to(DEV)
    p = Plan(n, DEV)
    for seed in (73, 74):  # the backward tables are rebuilt after every bfq_set_angles
        theta = synth.angles(n, "uniform", seed).to(DEV)
        p.set_angles(theta)
        dx, dth = p.backward(x, g)
        monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
        dx_gen, dth_gen = p.backward(x, g, dx_dtype=torch.float32)  # fp32 dx: one bf16 rounding between the two
        monkeypatch.delenv("BFQ_GENERIC_ONLY")
        check_rows_close(dx, to_f64(dx_gen), absmax_rows(g), "tuned vs generic dx")
        check_dtheta(dth, to_f64(dth_gen), "tuned vs generic dtheta")


def test_full_size_backward_n4096_sampled():
    wl = synth.WORKLOADS["learn4096"]
    rows = 65536  # a quarter of the learning batch keeps the oracle's share of the test to seconds
    theta = wl.theta(device=DEV)
    x = wl.x(device=DEV, n_rows=rows)
    g = wl.g(device=DEV, n_rows=rows)
    p = Plan(wl.n, DEV)
    p.set_angles(theta)
    dx = Guarded((rows, wl.n), torch.bfloat16, DEV)
    dth = Guarded((wl.L, wl.n // 2), torch.float32, DEV)
    p.backward(x, g, dx=dx.view, dtheta=dth.view)
    assert p.device_status() == 0 and dx.intact() and dth.intact()
    idx = _sample_rows(rows, 1024)
    ti = torch.from_numpy(idx).to(DEV)
    dx_ref, _ = oracle.backward(to_f64(theta), to_f64(x[ti]), to_f64(g[ti]))
    check_rows_close(dx.view[ti], dx_ref, absmax_rows(g[ti]), "learn4096 dx")
    # d-theta over all rows: linear in the rows, so the oracle's sum over 8 row blocks must match
    th64 = to_f64(theta)
    acc = np.zeros((wl.L, wl.n // 2))
    for r0 in range(0, rows, 8192):
        acc += oracle.backward(th64, to_f64(x[r0:r0 + 8192]), to_f64(g[r0:r0 + 8192]))[1]
    check_dtheta(dth.view, acc, "learn4096 dtheta")


# ---- tuned forward + INT2 for n = 8192 bf16 rows (two-CTA clusters) ---------------------------------------------
@pytest.mark.parametrize("rows", [1, 2, 3, 5, 73, 74 * 4 + 1, 1000])
@pytest.mark.parametrize("angle_kind", ["normal", "uniform"])
def test_tuned_n8192_int2_ragged_row_counts(rows, angle_kind):
    n = 8192
    theta = synth.angles(n, angle_kind, 80 + rows)
    if angle_kind == "uniform":
        theta[:, ::7] = math.pi / 2
        theta[:, 1::7] = -math.pi
        theta[:, 2::7] = math.pi
        theta[:, 3::7] = -math.pi / 2
        theta[:, 4::7] = 100.0
    x = synth.rows(rows, n, "laplace", 81 + rows, outliers=16, outlier_scale=100.0, dtype=torch.bfloat16)
    if rows >= 5:  # degenerate rows: zero, fp16-underflowing, fp16-saturating and subnormal scales
        x[0] = 0
        x[1] *= 1e-9
        x[2] *= 1e4
        x[3] *= 3e-8
    p = plan_for(n, theta)
    ld = n + 8
    xpad = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    xpad[:, :n] = x.to(DEV)
    codes = Guarded((rows, n // 4), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.forward_quant(xpad[:, :n], 2, codes=codes.view, scales=scales.view)
    assert p.device_status() == 0
    check_quant(codes.view, scales.view, oracle.forward(to_f64(theta), to_f64(x)), 2, f"tuned 8192 rows={rows}")
    assert codes.intact() and scales.intact()
    c2, s2 = p.forward_quant(xpad[:, :n], 2)
    assert torch.equal(c2, codes.view) and torch.equal(s2.view(torch.int16), scales.view.view(torch.int16))


def test_full_size_int2_n8192_and_fold_sampled():
    for name in ("act8192_int2", "fold8192_int2"):
        wl = synth.WORKLOADS[name]
        theta = wl.theta(device=DEV)
        x = wl.x(device=DEV)
        p = Plan(wl.n, DEV)
        p.set_angles(theta)
        if name.startswith("fold"):
            codes, scales, _ = p.fold_weights(x, 2)
        else:
            codes, scales = p.forward_quant(x, 2)
        assert p.device_status() == 0
        idx = _sample_rows(wl.n_rows, 1024)
        ti = torch.from_numpy(idx).to(DEV)
        y_ref = oracle.forward(to_f64(theta), to_f64(x[ti]))
        stats = check_quant(codes[ti], scales[ti], y_ref, 2, name)
        assert stats["scale_ulp_rows"] <= max(4, len(idx) // 100)
        del x, codes, scales


# ---- tuned inverse for n = 4096 and n = 8192 bf16 rows -------------------------------------------------------------
@pytest.mark.parametrize("rows", [1, 3, 147, 148 * 4 + 1, 1000])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("n", [4096, 8192])
def test_tuned_inverse(n, rows, out_dtype):
    theta = synth.angles(n, "uniform", 90 + rows)
    theta[:, ::7] = math.pi / 2
    theta[:, 1::7] = -math.pi
    theta[:, 3::7] = -math.pi / 2
    theta[:, 4::7] = 100.0
    y = synth.rows(rows, n, "student_t3", 91 + rows, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    ld = n + 8
    ypad = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    ypad[:, :n] = y.to(DEV)
    out = Guarded((rows, ld), out_dtype, DEV)
    p.inverse(ypad[:, :n], out=out.view[:, :n])
    assert p.device_status() == 0
    check_rows_close(out.view[:, :n], oracle.inverse(to_f64(theta), to_f64(y)), absmax_rows(y), f"tuned inverse rows={rows}")
    assert out.intact()
    # new angles on the same plan: the tables follow
    theta2 = synth.angles(n, "normal", 92 + rows)
    p.set_angles(theta2.to(DEV))
    x2 = p.inverse(y.to(DEV), out_dtype=out_dtype)
    check_rows_close(x2, oracle.inverse(to_f64(theta2), to_f64(y)), absmax_rows(y), "tuned inverse, second angle set")
    # round trip through the tuned-path forward of the generic kernels
    back = p.forward(x2.float(), out_dtype=torch.float32)
    check_rows_close(back, to_f64(y), 64 * absmax_rows(y), "round trip") if out_dtype == torch.float32 else None
    if n == 8192:
        # one half of the row on the three-shear tables, the other on the scaled ones
        assert p.stage_form() & 2 == 0
        theta3 = theta2.clone()
        theta3[3:7, :2048] = math.pi / 2  # four stages of the lower half: cosines of 4e-8 multiply up along every path
        p.set_angles(theta3.to(DEV))
        x3 = p.inverse(y.to(DEV), out_dtype=out_dtype)
        assert p.stage_form() & 2 == 2
        check_rows_close(x3, oracle.inverse(to_f64(theta3), to_f64(y)), absmax_rows(y), "tuned inverse, mixed forms")
        theta3[3:7, :2048], theta3[3:7, 2048:] = theta2[3:7, :2048], -math.pi / 2  # now only the upper half
        p.set_angles(theta3.to(DEV))
        x3 = p.inverse(y.to(DEV), out_dtype=out_dtype)
        assert p.stage_form() & 2 == 2
        check_rows_close(x3, oracle.inverse(to_f64(theta3), to_f64(y)), absmax_rows(y), "tuned inverse, mixed forms (upper)")


# ---- Walsh-Hadamard transform (the fixed rotation the paper compares with) and unquantized bf16 rows ---------------
@pytest.mark.parametrize("n", [16, 64, 256, 1024, 2048, 4096, 8192])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_hadamard_every_n(n, dtype):
    rows = 70 if n >= 2048 else 301
    x = synth.rows(rows, n, "student_t3", 100 + n, outliers=min(4, n // 4), outlier_scale=20.0, dtype=dtype)
    p = Plan(n, DEV)  # no angles needed
    ref = oracle.hadamard(to_f64(x))
    for out_dtype in (torch.float32, torch.bfloat16):
        out = Guarded((rows, n), out_dtype, DEV)
        p.hadamard(x.to(DEV), out=out.view)
        check_rows_close(out.view, ref, absmax_rows(x), f"hadamard n={n} {dtype}->{out_dtype}")
        assert out.intact()
    for bits in (2, 4, 8):
        codes, scales = p.hadamard_quant(x.to(DEV), bits)
        check_quant(codes, scales, ref, bits, f"hadamard_quant n={n} bits={bits}")
    assert p.device_status() == 0


@pytest.mark.parametrize("rows", [1, 5, 593, 1000])
@pytest.mark.parametrize("n", [4096, 8192])
def test_tuned_hadamard_and_bf16_rows(n, rows):
    theta = synth.angles(n, "uniform", 110 + rows)
    x = synth.rows(rows, n, "student_t3", 111 + rows, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    ld = n + 8
    xpad = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    xpad[:, :n] = x.to(DEV)
    xv = xpad[:, :n]
    y_ref, h_ref = oracle.forward(to_f64(theta), to_f64(x)), oracle.hadamard(to_f64(x))
    # learned butterfly, unquantized bf16 rows (the weight-only setting: activations stay 16-bit)
    out = Guarded((rows, ld), torch.bfloat16, DEV)
    p.forward(xv, out=out.view[:, :n])
    check_rows_close(out.view[:, :n], y_ref, absmax_rows(x), "tuned forward bf16")
    assert out.intact()
    # fixed Hadamard rotation, rows and INT4
    out = Guarded((rows, ld), torch.bfloat16, DEV)
    p.hadamard(xv, out=out.view[:, :n])
    check_rows_close(out.view[:, :n], h_ref, absmax_rows(x), "tuned hadamard bf16")
    assert out.intact()
    codes = Guarded((rows, n // 2), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.hadamard_quant(xv, 4, codes=codes.view, scales=scales.view)
    check_quant(codes.view, scales.view, h_ref, 4, "tuned hadamard INT4")
    assert codes.intact() and scales.intact() and p.device_status() == 0
    codes = Guarded((rows, n // 4), torch.uint8, DEV)
    p.hadamard_quant(xv, 2, codes=codes.view, scales=scales.view)
    check_quant(codes.view, scales.view, h_ref, 2, "tuned hadamard INT2")
    assert codes.intact() and scales.intact() and p.device_status() == 0


# ---- statistics riding on forward + quantize ---------------------------------------------------------------------
@pytest.mark.parametrize("n,rows,bits,dtype", [(256, 1000, 4, torch.float32), (4096, 333, 4, torch.bfloat16),
                                               (4096, 1, 4, torch.bfloat16), (4096, 1187, 4, torch.bfloat16),
                                               (4096, 77, 4, torch.float32),
                                               (8192, 70, 2, torch.bfloat16), (1024, 129, 8, torch.bfloat16)])
def test_forward_quant_stats(n, rows, bits, dtype):
    theta, x = make(n, rows, dtype, seed=120 + n)
    p = plan_for(n, theta)
    y_ref = oracle.forward(to_f64(theta), to_f64(x))
    codes, scales, hist, rowstats = p.forward_quant_stats(x.to(DEV), bits)
    check_quant(codes, scales, y_ref, bits, f"stats codes n={n}")
    # same codes and scales as the plain entry point (which may take a tuned kernel)
    c0, s0 = p.forward_quant(x.to(DEV), bits)
    assert torch.equal(s0.view(torch.int16), scales.view(torch.int16))
    got = oracle.unpack(codes.cpu().numpy(), bits)
    # the histogram is exact for the codes written, and close to the oracle's own (boundary cases aside)
    assert np.array_equal(hist.cpu().numpy(), oracle.code_histogram(got, bits))
    ref_hist = oracle.code_histogram(oracle.quantize(y_ref, bits)[0], bits)
    assert np.abs(hist.cpu().numpy() - ref_hist).sum() <= 2 * max(1, int(1e-4 * rows * n)) + 2 * n * 16
    assert oracle.uniformity_kl(hist.cpu().numpy()) == pytest.approx(oracle.uniformity_kl(ref_hist), abs=2e-3)
    np.testing.assert_allclose(to_f64(rowstats), oracle.row_moments(y_ref), rtol=2e-5)
    _, _, hist2, rs2 = p.forward_quant_stats(x.to(DEV), bits)
    assert torch.equal(hist, hist2) and torch.equal(rs2, rowstats)


# ---- rows in pinned host memory: chunked copies overlapped with the kernels -------------------------------------------
@pytest.mark.parametrize("rows,chunks", [(1000, 8), (5, 8), (4096, 3)])
def test_host_pipeline_matches_the_resident_call(rows, chunks):
    from paper_2509_09679_b200 import HostForwardQuant
    theta, x = make(4096, rows, torch.bfloat16, seed=77)
    p = plan_for(4096, theta)
    c_ref, s_ref = p.forward_quant(x.to(DEV), 4)
    x_host = x.pin_memory()
    c_host = torch.zeros((rows, 2048), dtype=torch.uint8).pin_memory()
    s_host = torch.zeros((rows,), dtype=torch.float16).pin_memory()
    pipe = HostForwardQuant(p, rows, 4, chunks=chunks)
    for _ in range(2):  # second call reuses the buffers and events
        c_host.zero_()
        pipe(x_host, c_host, s_host, before=lambda: p.set_angles(theta.to(DEV)))
        torch.cuda.synchronize()
        assert torch.equal(c_host, c_ref.cpu()) and torch.equal(s_host.view(torch.int16), s_ref.cpu().view(torch.int16))
    assert p.device_status() == 0


@pytest.mark.parametrize("n,rows,bits,dtype", [(256, 77, 8, torch.float32), (4096, 300, 2, torch.float32),
                                               (8192, 41, 2, torch.bfloat16)])
def test_host_entry_point_other_shapes(n, rows, bits, dtype):
    """bfq_forward_quant_host through the binding: fp32 rows, a padded leading dimension on the host, chunks that do not
    divide the row count, generic and tuned kernels; results equal the device-resident call bit for bit."""
    theta, x = make(n, rows, dtype, seed=91)
    p = plan_for(n, theta)
    c_ref, s_ref = p.forward_quant(x.to(DEV), bits)
    x_host = torch.zeros((rows, n + 16), dtype=dtype).pin_memory()
    x_host[:, :n] = x
    c_host = torch.zeros((rows, n * bits // 8), dtype=torch.uint8).pin_memory()
    s_host = torch.zeros((rows,), dtype=torch.float16).pin_memory()
    ws = torch.empty((p.forward_quant_host_workspace(dtype, bits, 24),), dtype=torch.uint8, device=DEV)
    p.forward_quant_host(x_host[:, :n], bits, c_host, s_host, ws)
    torch.cuda.synchronize()
    assert torch.equal(c_host, c_ref.cpu()) and torch.equal(s_host.view(torch.int16), s_ref.cpu().view(torch.int16))
    with pytest.raises(BfqError):  # a workspace too small for two chunks of eight rows
        p.forward_quant_host(x_host[:, :n], bits, c_host, s_host, ws[:64])
    assert p.device_status() == 0


@pytest.mark.parametrize("rows", [1, 3, 130, 593, 1001])
@pytest.mark.parametrize("n,bits", [(4096, 2), (4096, 8), (8192, 4), (8192, 8)])
def test_tuned_kernels_other_bit_widths(rows, n, bits, monkeypatch):
    theta, x = make(n, rows, torch.bfloat16, seed=300 + rows)
    if rows >= 130:  # degenerate rows: zero, tiny (subnormal scale) and huge (saturated scale)
        xs = x.float()
        xs[1] = 0.0
        xs[2] *= 1e-8
        xs[3] *= 1e30
        x = xs.to(torch.bfloat16)
    p = plan_for(n, theta)
    y_ref = oracle.forward(to_f64(theta), to_f64(x))
    codes = Guarded((rows, n * bits // 8), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.forward_quant(x.to(DEV), bits, codes=codes.view, scales=scales.view)
    assert p.device_status() == 0 and codes.intact() and scales.intact()
    check_quant(codes.view, scales.view, y_ref, bits, f"tuned n={n} INT{bits}")
    monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
    c_g, s_g = p.forward_quant(x.to(DEV), bits)
    monkeypatch.delenv("BFQ_GENERIC_ONLY")
    assert (s_g.view(torch.int16).int() - scales.view.view(torch.int16).int()).abs().max().item() <= 1
    assert (c_g != codes.view).float().mean().item() < 1e-3


@pytest.mark.parametrize("rows", [1, 2, 3, 75, 297, 1000])
def test_tuned_n8192_bf16_rows(rows):
    """y = Q x in bf16 at n = 8192 (weight-only setting: 16-bit activations) on the cluster kernel, padded leading dimensions."""
    theta, x = make(8192, rows, torch.bfloat16, seed=500 + rows)
    p = plan_for(8192, theta)
    xs = torch.zeros((rows, 8192 + 64), dtype=torch.bfloat16, device=DEV)
    xs[:, :8192] = x.to(DEV)
    ybuf = Guarded((rows, 8192 + 128), torch.bfloat16, DEV)
    y = ybuf.view[:, :8192]
    p.forward(xs[:, :8192], out=y)
    assert p.device_status() == 0 and ybuf.intact()
    assert (ybuf.view[:, 8192:].view(torch.int16) == torch.tensor(0xA5A5, dtype=torch.uint16).view(torch.int16).item()).all()
    check_rows_close(y, oracle.forward(to_f64(theta), to_f64(x)), absmax_rows(x), "tuned n=8192 bf16 rows")


def test_fold_weights_n4096_int2_on_the_tuned_kernel():
    """2-bit weights of an n = 4096 layer (the paper's W2 setting at the 7B shape): W Q^T through the tuned kernel's INT2
    epilogue, and computational invariance of the quantized product against the oracle's own."""
    n, m = 4096, 300
    theta = synth.angles(n, "normal", 31)
    W = synth.rows(m, n, "normal", 32, scale=0.02, dtype=torch.bfloat16)
    x = synth.rows(24, n, "student_t3", 33, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    th64 = to_f64(theta)
    codes, scales, _ = p.fold_weights(W.to(DEV), 2)
    WQt_ref = oracle.forward(th64, to_f64(W))
    check_quant(codes, scales, WQt_ref, 2, "fold n=4096 INT2")
    Qx = to_f64(p.forward(x.to(DEV), out_dtype=torch.float32))
    ref = to_f64(W) @ to_f64(x).T
    o_codes, o_scales = oracle.quantize(WQt_ref, 2)
    err_ref = np.linalg.norm(oracle.dequantize(o_codes, o_scales) @ oracle.forward(th64, to_f64(x)).T - ref)
    deq = oracle.dequantize(oracle.unpack(codes.cpu().numpy(), 2), scales.cpu().view(torch.int16).numpy().view(np.uint16))
    assert abs(np.linalg.norm(deq @ Qx.T - ref) - err_ref) <= 1e-3 * err_ref
    assert p.device_status() == 0


@pytest.mark.parametrize("n,bits,m", [(4096, 2, 293), (4096, 4, 37), (4096, 8, 5), (8192, 2, 151), (8192, 4, 9)])
def test_fold_weights_with_rotated_rows_on_the_tuned_kernels(n, bits, m):
    """bfq_fold_weights that also keeps W Q^T in bf16: codes, scales and rotated rows come from one pass of the tuned
    kernels and must agree with the oracle like the two outputs do separately; the generic kernel gives the same codes."""
    theta = synth.angles(n, "normal", 41)
    W = synth.rows(m, n, "normal", 42, scale=0.02, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    ref = oracle.forward(to_f64(theta), to_f64(W))
    codes, scales, rot = p.fold_weights(W.to(DEV), bits, want_rotated=True)
    assert rot.dtype == torch.bfloat16
    check_quant(codes, scales, ref, bits, f"fold + rows n={n} INT{bits}: codes")
    check_rows_close(rot, ref, absmax_rows(W), f"fold + rows n={n} INT{bits}: rows")
    codes2, scales2, _ = p.fold_weights(W.to(DEV), bits)
    assert torch.equal(codes, codes2) and torch.equal(scales.view(torch.int16), scales2.view(torch.int16))
    assert p.device_status() == 0


@pytest.mark.parametrize("rows", [1, 3, 130, 593, 1001])
@pytest.mark.parametrize("bits", [0, 2, 4, 8])
@pytest.mark.parametrize("n", [4096, 8192])
def test_tuned_fp32_rows(n, rows, bits, monkeypatch):
    """fp32 rows at n = 4096 / 8192 take the tuned kernels (fp32 tensor map, one input slot per row group): rotated rows
    in fp32 (bits = 0) and codes of every width against the oracle, degenerate rows included, a padded leading dimension,
    and agreement with the generic kernels."""
    theta, x = make(n, rows, torch.float32, seed=500 + rows + bits)
    if rows >= 130:  # zero, tiny (subnormal scale) and huge (saturated scale) rows
        x[1] = 0.0
        x[2] *= 1e-8
        x[3] *= 1e30
    p = plan_for(n, theta)
    xpad = torch.zeros((rows, n + 8), dtype=torch.float32, device=DEV)
    xpad[:, :n] = x.to(DEV)
    xv = xpad[:, :n]
    y_ref = oracle.forward(to_f64(theta), to_f64(x))
    if bits == 0:
        amax = np.abs(to_f64(x)).max(axis=1)
        keep = (amax < 1e20) & (amax > 0)  # the absolute tolerance means nothing for the 1e30 row
        out = Guarded((rows, n), torch.float32, DEV)
        p.forward(xv, out=out.view)
        assert out.intact() and p.device_status() == 0
        if rows >= 130:
            assert not out.view[1].any()  # the zero row stays zero
        check_rows_close(out.view[torch.from_numpy(keep).to(DEV)], y_ref[keep], absmax_rows(x)[keep], "tuned fp32 rows")
        if n == 4096:  # the tuned inverse reads fp32 rows the same way
            inv = Guarded((rows, n), torch.float32, DEV)
            p.inverse(xv, out=inv.view)
            assert inv.intact() and p.device_status() == 0
            xi_ref = oracle.inverse(to_f64(theta), to_f64(x))
            check_rows_close(inv.view[torch.from_numpy(keep).to(DEV)], xi_ref[keep], absmax_rows(x)[keep], "tuned fp32 inverse")
        return
    codes = Guarded((rows, n * bits // 8), torch.uint8, DEV)
    scales = Guarded((rows,), torch.float16, DEV)
    p.forward_quant(xv, bits, codes=codes.view, scales=scales.view)
    assert p.device_status() == 0 and codes.intact() and scales.intact()
    check_quant(codes.view, scales.view, y_ref, bits, f"tuned fp32 n={n} INT{bits}")
    monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
    c_g, s_g = p.forward_quant(xv, bits)
    monkeypatch.delenv("BFQ_GENERIC_ONLY")
    assert (s_g.view(torch.int16).int() - scales.view.view(torch.int16).int()).abs().max().item() <= 1
    assert (c_g != codes.view).float().mean().item() < 1e-3


@pytest.mark.parametrize("rows", [1, 2, 3, 75, 297, 1001])
@pytest.mark.parametrize("angle_kind", ["normal", "uniform"])
def test_tuned_backward_n8192_ragged_row_counts(rows, angle_kind, monkeypatch):
    """n = 8192 bf16 rows: stage 12's sums come from the forward cluster kernel, stages 0 .. 11 and dx from two launches of
    the n = 4096 backward kernel (one per half of the elements): everything against the oracle, a padded leading
    dimension, the same bits when run again, and agreement with the generic kernel."""
    n = 8192
    theta = synth.angles(n, angle_kind, 80 + rows)
    if angle_kind == "uniform":
        theta[:, ::7] = math.pi / 2
        theta[:, 1::7] = -math.pi
        theta[:, 4::7] = 100.0
    x = synth.rows(rows, n, "laplace", 81 + rows, outliers=16, outlier_scale=100.0, dtype=torch.bfloat16)
    g = synth.rows(rows, n, "normal", 82 + rows, dtype=torch.bfloat16)
    p = plan_for(n, theta)
    ld = n + 8
    xpad = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    gpad = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    xpad[:, :n] = x.to(DEV)
    gpad[:, :n] = g.to(DEV)
    dxbuf = Guarded((rows, ld), torch.bfloat16, DEV)
    dth = Guarded((p.L, n // 2), torch.float32, DEV)
    p.backward(xpad[:, :n], gpad[:, :n], dx=dxbuf.view[:, :n], dtheta=dth.view)
    assert p.device_status() == 0
    dx_ref, dth_ref = oracle.backward(to_f64(theta), to_f64(x), to_f64(g))
    check_rows_close(dxbuf.view[:, :n], dx_ref, absmax_rows(g), f"n=8192 dx rows={rows}")
    check_dtheta(dth.view, dth_ref, f"n=8192 dtheta rows={rows}")
    assert dxbuf.intact() and dth.intact()
    assert (dxbuf.view[:, n:].contiguous().view(torch.int16) == torch.tensor(0xA5A5, dtype=torch.uint16).view(torch.int16)).all()
    _, dth2 = p.backward(xpad[:, :n], gpad[:, :n], want_dx=False)
    assert torch.equal(dth2, dth.view)
    monkeypatch.setenv("BFQ_GENERIC_ONLY", "1")
    dx_gen, dth_gen = p.backward(xpad[:, :n], gpad[:, :n], dx_dtype=torch.float32)
    monkeypatch.delenv("BFQ_GENERIC_ONLY")
    check_rows_close(dxbuf.view[:, :n], to_f64(dx_gen), absmax_rows(g), "n=8192 tuned vs generic dx")
    check_dtheta(dth.view, to_f64(dth_gen), "n=8192 tuned vs generic dtheta")
