"""Pins for the CPU oracle: every check compares it with something the paper or the
mathematics fixes (printed matrices, closed forms, invariants, brute force, finite
differences, hand-worked examples), never with itself or with the CUDA path."""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(20250909)


def rand_theta(n, rng=RNG, lo=-math.pi, hi=math.pi):
    L = n.bit_length() - 1
    return rng.uniform(lo, hi, size=(L, n // 2))


def dense_Q(theta):
    """Brute force: Q = B_L ... B_2 B_1 as an explicit product of dense layer matrices."""
    L, half = theta.shape
    n = 2 * half
    Q = np.eye(n)
    for s in range(L):
        Q = oracle.dense_stage(n, s, theta[s]) @ Q
    return Q


# ---- P1: the printed n = 8 layer matrices (appendix example) -------------------------
def test_n8_layer_matrices_match_the_printed_ones():
    theta = rand_theta(8)
    expect = np.zeros((3, 8, 8))
    with open(os.path.join(GOLDEN, "n8_layers.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            layer, row, col, sign, func, j = line.split()
            t = theta[int(layer) - 1][int(j) - 1]
            v = math.cos(t) if func == "cos" else math.sin(t)
            expect[int(layer) - 1, int(row), int(col)] = v if sign == "+" else -v
    for s in range(3):
        np.testing.assert_allclose(oracle.dense_stage(8, s, theta[s]), expect[s], rtol=0, atol=1e-15)
    # and the fast application applies layer 1 first: y = B3 (B2 (B1 x))
    x = RNG.standard_normal(8)
    np.testing.assert_allclose(oracle.forward(theta, x), expect[2] @ (expect[1] @ (expect[0] @ x)),
                               atol=1e-14)


# ---- P2: orthogonality by construction ------------------------------------------------
@pytest.mark.parametrize("n", [2, 4, 8, 16, 64])
def test_QtQ_is_identity_and_norm_is_preserved(n):
    theta = rand_theta(n)
    Q = dense_Q(theta)
    np.testing.assert_allclose(Q.T @ Q, np.eye(n), atol=1e-12)
    x = RNG.standard_normal((5, n))
    y = oracle.forward(theta, x)
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)


# ---- P3: identity initialisation ---------------------------------------------------------
@pytest.mark.parametrize("n", [2, 8, 64, 256])
def test_zero_angles_give_identity(n):
    theta = np.zeros((n.bit_length() - 1, n // 2))
    x = RNG.standard_normal((3, n))
    assert np.array_equal(oracle.forward(theta, x), x)
    assert np.array_equal(oracle.inverse(theta, x), x)


# ---- P4: Hadamard special case: theta = pi/4 ----------------------------------------------
@pytest.mark.parametrize("n", [2, 4, 8, 64])
def test_pi_over_4_is_hadamard_times_sign_diagonal(n):
    theta = np.full((n.bit_length() - 1, n // 2), math.pi / 4)
    Q = oracle.forward(theta, np.eye(n)).T  # row k of forward(I) is Q e_k = column k of Q
    i = np.arange(n)[:, None]
    j = np.arange(n)[None, :]
    pop = np.vectorize(lambda v: bin(v).count("1"))
    closed = (-1.0) ** (pop(i & j) + pop(j)) / math.sqrt(n)  # H_2 = G(pi/4) diag(1,-1)
    np.testing.assert_allclose(Q, closed, atol=1e-14)
    # Sylvester Hadamard built by the recursive definition, times D = diag((-1)^popcount(j))
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]]) / math.sqrt(2)
    D = np.diag((-1.0) ** pop(np.arange(n)))
    np.testing.assert_allclose(Q, H @ D, atol=1e-14)
    # coherence attains 1/sqrt(n)
    off = np.abs(Q - np.diag(np.diag(Q)))
    assert abs(off.max() - 1 / math.sqrt(n)) < 1e-14


def test_coherence_at_n4096_is_the_welch_bound():
    n = 4096
    theta = np.full((12, n // 2), math.pi / 4)
    rows = np.zeros((64, n))
    cols = RNG.choice(n, size=64, replace=False)
    rows[np.arange(64), cols] = 1.0
    y = oracle.forward(theta, rows)
    np.testing.assert_allclose(np.abs(y), 0.015625, atol=1e-15)  # 1/sqrt(4096) = 1.56e-2


# ---- P5: stage-uniform angles give a Kronecker product of 2x2 rotations --------------------
@pytest.mark.parametrize("n", [4, 16, 64])
def test_stage_uniform_angles_closed_form(n):
    L = n.bit_length() - 1
    per_stage = RNG.uniform(-math.pi, math.pi, size=L)
    theta = np.repeat(per_stage[:, None], n // 2, axis=1)
    Q = oracle.forward(theta, np.eye(n)).T
    expect = np.ones((n, n))
    for s in range(L):
        c, sn = math.cos(per_stage[s]), math.sin(per_stage[s])
        G = np.array([[c, -sn], [sn, c]])
        bi = (np.arange(n) >> s) & 1
        expect *= G[bi[:, None], bi[None, :]]
    np.testing.assert_allclose(Q, expect, atol=1e-13)


# ---- P6: fast application equals the dense product (brute force) ---------------------------
@pytest.mark.parametrize("n", [2, 4, 8, 16, 32, 64])
def test_fast_equals_dense_product(n):
    theta = rand_theta(n)
    Q = dense_Q(theta)
    x = RNG.standard_normal((7, n))
    np.testing.assert_allclose(oracle.forward(theta, x), x @ Q.T, atol=1e-12)
    np.testing.assert_allclose(oracle.inverse(theta, x), x @ Q, atol=1e-12)


def test_stage_order_matters_and_stride_one_is_first():
    # With distinct angles the layers do not commute: the opposite order gives another matrix.
    theta = rand_theta(8)
    B = [oracle.dense_stage(8, s, theta[s]) for s in range(3)]
    assert not np.allclose(B[2] @ B[1] @ B[0], B[0] @ B[1] @ B[2])
    x = RNG.standard_normal(8)
    np.testing.assert_allclose(oracle.forward(theta, x), B[2] @ B[1] @ B[0] @ x, atol=1e-14)


# ---- P7: round trip ---------------------------------------------------------------------------
@pytest.mark.parametrize("n", [2, 16, 256, 4096])
def test_inverse_of_forward_is_identity(n):
    theta = rand_theta(n)
    x = RNG.standard_normal((4, n)) * 10
    np.testing.assert_allclose(oracle.inverse(theta, oracle.forward(theta, x)), x, atol=1e-11)
    np.testing.assert_allclose(oracle.forward(theta, oracle.inverse(theta, x)), x, atol=1e-11)


# ---- P8: gradients ----------------------------------------------------------------------------
@pytest.mark.parametrize("n", [2, 4, 8, 16])
def test_dtheta_matches_central_finite_differences(n):
    theta = rand_theta(n)
    rows = 3
    x = RNG.standard_normal((rows, n))
    g = RNG.standard_normal((rows, n))
    dx, dth = oracle.backward(theta, x, g)
    h = 1e-6
    fd = np.zeros_like(theta)
    for s in range(theta.shape[0]):
        for j in range(theta.shape[1]):
            tp = theta.copy()
            tp[s, j] += h
            tm = theta.copy()
            tm[s, j] -= h
            fd[s, j] = (np.sum(g * oracle.forward(tp, x)) - np.sum(g * oracle.forward(tm, x))) / (2 * h)
    np.testing.assert_allclose(dth, fd, atol=1e-7)
    # dx = Q^T g
    np.testing.assert_allclose(dx, g @ dense_Q(theta), atol=1e-12)
    np.testing.assert_allclose(dx, oracle.inverse(theta, g), atol=1e-12)


def test_single_rotation_gradient_is_the_printed_derivative():
    # n = 2: dL/dtheta = g^T (dG/dtheta) x with dG/dtheta = [[-sin, -cos], [cos, -sin]]
    t = 0.37
    x = np.array([[1.3, -0.4]])
    g = np.array([[0.2, 0.9]])
    dG = np.array([[-math.sin(t), -math.cos(t)], [math.cos(t), -math.sin(t)]])
    _, dth = oracle.backward(np.array([[t]]), x, g)
    assert abs(dth[0, 0] - (g @ dG @ x.T)[0, 0]) < 1e-15


@pytest.mark.parametrize("n", [8, 64, 256])
def test_adjoint_identity_and_norm_gradient(n):
    theta = rand_theta(n)
    x = RNG.standard_normal((6, n))
    g = RNG.standard_normal((6, n))
    y = oracle.forward(theta, x)
    dx, dth = oracle.backward(theta, x, g)
    # <g, Qx> = <Q^T g, x>
    np.testing.assert_allclose(np.sum(g * y), np.sum(dx * x), rtol=1e-12)
    # L = 1/2 |Qx|^2 is constant in theta: g = y gives dtheta = 0 and dx = x
    dx2, dth2 = oracle.backward(theta, x, y)
    np.testing.assert_allclose(dth2, 0, atol=1e-11)
    np.testing.assert_allclose(dx2, x, atol=1e-12)
    # input form (used by the oracle) equals the output form  g_hi*z'_lo - g_lo*z'_hi
    L = theta.shape[0]
    out_form = np.zeros_like(theta)
    z = y.copy()
    gb = g.copy()
    for s in reversed(range(L)):
        h = 1 << s
        j = np.arange(n // 2)
        lo = ((j >> s) << (s + 1)) | (j & (h - 1))
        hi = lo + h
        out_form[s] = np.sum(gb[:, hi] * z[:, lo] - gb[:, lo] * z[:, hi], axis=0)
        Bs = oracle.dense_stage(n, s, theta[s])
        z = z @ Bs      # row-vector form of B^T z
        gb = gb @ Bs
    np.testing.assert_allclose(dth, out_form, atol=1e-10)


def test_dtheta_is_summed_over_rows_and_thread_count_independent():
    n = 64
    theta = rand_theta(n)
    x = RNG.standard_normal((200, n))
    g = RNG.standard_normal((200, n))
    _, dth = oracle.backward(theta, x, g)
    acc = np.zeros_like(theta)
    for r in range(0, 200, 50):
        acc += oracle.backward(theta, x[r:r + 50], g[r:r + 50])[1]
    np.testing.assert_allclose(dth, acc, atol=1e-10)


# ---- P9: counts the paper prints ------------------------------------------------------------------
def test_parameter_counts():
    for n, angles in [(128, 448), (4096, 24576)]:
        L = n.bit_length() - 1
        assert L * n // 2 == angles
        assert rand_theta(n).shape == (L, n // 2)
    assert 24576 * 2 * 2 == 98304  # (cos, sin) pairs in fp16 at n = 4096
    # 5120 = 40 x 128: 780 Cayley parameters + 448 angles
    assert 40 * 39 // 2 + 448 == 1228


# ---- P10: quantizer ----------------------------------------------------------------------------------
def _golden_quant():
    with open(os.path.join(GOLDEN, "quant_examples.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, ys, sc, codes, packed = [p.strip() for p in line.split("|")]
            yield (int(bits), np.array([float(v) for v in ys.split()]), int(sc, 16),
                   np.array([int(v) for v in codes.split()], dtype=np.int8),
                   np.array([int(v, 16) for v in packed.split()], dtype=np.uint8))


def test_quantizer_hand_worked_examples():
    for bits, y, sc, codes, packed in _golden_quant():
        c, s = oracle.quantize(y[None, :], bits)
        assert int(s[0]) == sc, (bits, hex(int(s[0])))
        assert np.array_equal(c[0], codes), (bits, c[0])
        assert np.array_equal(oracle.pack(c, bits)[0], packed)
        assert np.array_equal(oracle.unpack(packed[None, :], bits)[0], codes)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quantizer_properties(bits):
    n, rows = 256, 64
    qmax = 2 ** (bits - 1) - 1
    y = RNG.standard_t(3, size=(rows, n)) * RNG.uniform(0.01, 100, size=(rows, 1))
    codes, s16, pre = oracle.quantize(y, bits, want_prequant=True)
    s = oracle.f16_bits_to_f64(s16)
    amax = np.abs(y).max(axis=1)
    # scale is amax/qmax to fp16 accuracy (relative 2^-11)
    np.testing.assert_allclose(s, amax / qmax, rtol=2.0 ** -11)
    assert codes.min() >= -(2 ** (bits - 1)) and codes.max() <= qmax
    # error bound s/2 wherever no clipping happened
    deq = oracle.dequantize(codes, s16)
    unclipped = np.abs(pre) <= qmax + 0.5
    assert np.all(np.abs(deq - y)[unclipped] <= s[:, None].repeat(n, 1)[unclipped] * (0.5 + 1e-6))
    # the arg-max element maps to +-qmax
    k = np.abs(y).argmax(axis=1)
    assert np.array_equal(np.abs(codes[np.arange(rows), k]), np.full(rows, qmax))
    # idempotent: re-quantising the dequantised row with the same scale returns the codes
    c2, _ = oracle.quantize(deq, bits, scale_in=s16)
    assert np.array_equal(c2, codes)
    # pack / unpack round trip
    assert np.array_equal(oracle.unpack(oracle.pack(codes, bits), bits), codes)
    # an independent numpy statement of the same quantizer
    sf = (amax.astype(np.float32) / np.float32(qmax)).astype(np.float16)
    assert np.array_equal(sf.view(np.uint16), s16)
    ref = np.clip(np.rint((y / sf.astype(np.float64)[:, None]).astype(np.float32)), -(qmax + 1), qmax)
    assert np.array_equal(ref.astype(np.int8), codes)


def test_fp16_rounding_matches_numpy_float16():
    vals = np.concatenate([
        RNG.uniform(-70000, 70000, 2000), RNG.uniform(-1, 1, 2000) * 1e-4,
        RNG.uniform(-1, 1, 2000) * 1e-7, np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9,
                                                    2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25, 2.0 ** -14]),
        (np.arange(1, 2049) + 0.5) * 2.0 ** -3,   # exact ties in the normal range
        (np.arange(0, 1024) + 0.5) * 2.0 ** -24,  # exact ties in the subnormal range
    ]).astype(np.float32)
    got = np.array([oracle.f32_to_f16_bits(float(v)) for v in vals], dtype=np.uint16)
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16)
    big = np.isinf(ref)
    ref_bits = ref.view(np.uint16).copy()
    ref_bits[big] = np.where(vals[big] > 0, 0x7BFF, 0xFBFF)  # saturate instead of inf
    assert np.array_equal(got, ref_bits)
    back = np.array([oracle.lib().orc_f16_to_f64(int(b)) for b in got[~big]])
    assert np.array_equal(back, ref[~big].astype(np.float64))


def test_clipping_range_is_asymmetric_twos_complement():
    # clip(round(x/s), -2^(b-1), 2^(b-1)-1) with a given scale of 1.0 (fp16 0x3C00)
    y = np.array([[20.0, -20.0, 3.0, -8.4, 7.5, -7.5, 8.5, -8.5]])
    one = np.array([0x3C00], dtype=np.uint16)
    c4, _ = oracle.quantize(y, 4, scale_in=one)
    assert c4[0].tolist() == [7, -8, 3, -8, 7, -8, 7, -8]
    c2, _ = oracle.quantize(y, 2, scale_in=one)
    assert c2[0].tolist() == [1, -2, 1, -2, 1, -2, 1, -2]
    c8, _ = oracle.quantize(y * 20, 8, scale_in=one)
    assert c8[0].tolist() == [127, -128, 60, -128, 127, -128, 127, -128]


def test_zero_and_tiny_rows():
    y = np.zeros((2, 16))
    y[1, 3] = 1e-9  # scale underflows to fp16 zero: all codes zero
    codes, s16 = oracle.quantize(y, 4)
    assert np.array_equal(s16, np.zeros(2, dtype=np.uint16))
    assert not codes.any()


# ---- P11: fold invariance (W Q^T)(Q x) = W x ------------------------------------------------------------
@pytest.mark.parametrize("n", [16, 256])
def test_fold_is_forward_on_weight_rows(n):
    theta = rand_theta(n)
    W = RNG.standard_normal((12, n)) * 0.02
    x = RNG.standard_normal((9, n))
    _, _, WQt = oracle.fold_weights(theta, W, 2, want_y=True)
    Qx = oracle.forward(theta, x)
    np.testing.assert_allclose(WQt @ Qx.T, W @ x.T, atol=1e-10)
    # using Q^T w instead would break the invariance
    wrong = oracle.inverse(theta, W)
    assert not np.allclose(wrong @ Qx.T, W @ x.T, atol=1e-6)
    # and W Q^T as a dense product
    np.testing.assert_allclose(WQt, W @ dense_Q(theta).T, atol=1e-12)


def test_forward_quant_is_forward_then_quantize():
    n = 64
    theta = rand_theta(n)
    x = RNG.standard_t(3, size=(10, n))
    packed, s16, y = oracle.forward_quant(theta, x, 4, want_y=True)
    np.testing.assert_array_equal(y, oracle.forward(theta, x))
    codes, s2 = oracle.quantize(y, 4)
    assert np.array_equal(s2, s16) and np.array_equal(oracle.pack(codes, 4), packed)


def test_bf16_widening_is_exact():
    import torch

    t = torch.randn(1000, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    bits = t.view(torch.int16).numpy()
    assert np.array_equal(oracle.bf16_bits_to_f64(bits), t.to(torch.float64).numpy())


# ---- Hadamard transform (the fixed rotation of Sec. 3.1.1) -----------------------------------------------
def test_hadamard_is_the_kronecker_power_of_h2_and_relates_to_the_pi_over_4_butterfly():
    h2 = np.array([[1.0, 1.0], [1.0, -1.0]]) / math.sqrt(2.0)
    for n in (2, 4, 8, 64):
        H = np.array([[1.0]])
        for _ in range(n.bit_length() - 1):
            H = np.kron(h2, H)  # H_2n = 1/sqrt(2) [[H, H], [H, -H]]
        got = oracle.hadamard(np.eye(n)).T  # row i of the result is H e_i, i.e. column i of H
        np.testing.assert_allclose(got, H, atol=1e-14)
        np.testing.assert_allclose(np.abs(got), 1.0 / math.sqrt(n), atol=1e-14)  # coherence 1/sqrt(n)
        np.testing.assert_allclose(got @ got.T, np.eye(n), atol=1e-13)
        # theorem "Hadamard is a butterfly": all theta = pi/4 gives Q = H_n D, D_jj = (-1)^popcount(j)
        theta = np.full((n.bit_length() - 1, n // 2), math.pi / 4)
        x = RNG.standard_normal((5, n))
        D = np.array([(-1.0) ** bin(j).count("1") for j in range(n)])
        np.testing.assert_allclose(oracle.forward(theta, x), oracle.hadamard(x * D), atol=1e-13)
    x = RNG.standard_normal((3, 4096))
    y = oracle.hadamard(x)
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-13)
    np.testing.assert_allclose(oracle.hadamard(y), x, atol=1e-12)  # H is symmetric and orthogonal


# ---- statistics of rotated rows: code histogram, uniformity divergence, moments ---------------------------
def test_uniformity_kl_and_moments_closed_forms():
    assert oracle.uniformity_kl(np.full(16, 7)) == pytest.approx(0.0, abs=1e-15)          # uniform bins
    one = np.zeros(16)
    one[3] = 5
    assert oracle.uniformity_kl(one) == pytest.approx(math.log(16.0), rel=1e-15)          # all mass in one bin
    two = np.zeros(4)
    two[[0, 2]] = 1
    assert oracle.uniformity_kl(two) == pytest.approx(math.log(2.0), rel=1e-15)           # half of the bins
    codes = np.array([[-8, 7, 0, 0], [1, -1, 7, -8]])
    h = oracle.code_histogram(codes, 4)
    assert h.sum() == 8 and h[0] == 2 and h[15] == 2 and h[8] == 2 and h[9] == 1 and h[7] == 1
    # moments: +-1 rows have kurtosis exactly 1; a rotation preserves sum y^2
    pm = np.where(RNG.random((3, 64)) < 0.5, -1.0, 1.0)
    m = oracle.row_moments(pm)
    np.testing.assert_allclose(64 * m[:, 1] / m[:, 0] ** 2, 1.0, rtol=1e-15)
    theta, x = rand_theta(64), RNG.standard_normal((4, 64))
    np.testing.assert_allclose(oracle.row_moments(oracle.forward(theta, x))[:, 0], (x * x).sum(axis=1), rtol=1e-12)
    g = RNG.standard_normal((1, 1 << 20))
    mg = oracle.row_moments(g)[0]
    assert (1 << 20) * mg[1] / mg[0] ** 2 == pytest.approx(3.0, abs=0.03)                 # Gaussian kurtosis


# ---- composite transform for non-power-of-2 sizes: Cayley factor (x) butterfly (Sec. 3.3) --------------------
def test_cayley_and_kronecker_composite():
    # 2 x 2 by hand: A = [[0, a], [-a, 0]]; (I - A)(I + A)^-1 = [[1 - a^2, -2a], [2a, 1 - a^2]] / (1 + a^2),
    # the rotation by 2 atan(a)
    a = 0.37
    Q = oracle.cayley([a], 2)
    np.testing.assert_allclose(Q, np.array([[1 - a * a, -2 * a], [2 * a, 1 - a * a]]) / (1 + a * a), atol=1e-15)
    phi = 2.0 * math.atan(a)
    np.testing.assert_allclose(Q, [[math.cos(phi), -math.sin(phi)], [math.sin(phi), math.cos(phi)]], atol=1e-15)
    np.testing.assert_allclose(oracle.cayley(np.zeros(780), 40), np.eye(40), atol=0)        # A = 0 gives I
    p = RNG.standard_normal(780) * 0.2
    Q1 = oracle.cayley(p, 40)
    np.testing.assert_allclose(Q1.T @ Q1, np.eye(40), atol=1e-13)                           # orthogonal by construction
    assert abs(np.linalg.det(Q1) - 1.0) < 1e-12
    assert 780 + 7 * 64 == 1228 and round(5120 * 5120 / 1228) == 21347                      # the paper's parameter count
    # (Q1 kron Q2) x by brute force on a small case, and orthogonality of the composite
    n1, n2 = 5, 8
    Q1s = oracle.cayley(RNG.standard_normal(n1 * (n1 - 1) // 2), n1)
    th2 = rand_theta(n2)
    K = np.kron(Q1s, dense_Q(th2))
    x = RNG.standard_normal((6, n1 * n2))
    np.testing.assert_allclose(oracle.composite_forward(Q1s, th2, x), x @ K.T, atol=1e-13)
    np.testing.assert_allclose(K.T @ K, np.eye(n1 * n2), atol=1e-13)
    y = oracle.composite_forward(Q1, rand_theta(128), RNG.standard_normal((2, 5120)))
    assert y.shape == (2, 5120)
    # the inverse is the transpose of the Kronecker matrix, undoes the forward map and is its adjoint
    z = RNG.standard_normal((6, n1 * n2))
    np.testing.assert_allclose(oracle.composite_inverse(Q1s, th2, z), z @ K, atol=1e-13)
    np.testing.assert_allclose(oracle.composite_inverse(Q1s, th2, oracle.composite_forward(Q1s, th2, x)), x, atol=1e-13)
    assert abs(np.sum(oracle.composite_forward(Q1s, th2, x) * z) - np.sum(x * oracle.composite_inverse(Q1s, th2, z))) < 1e-12
