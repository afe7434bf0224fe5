"""CPU oracle (test infrastructure) for the butterfly-rotation + quantization path.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It wraps ``bfq_oracle.c`` (plain C, fp64) through ctypes and never touches
the CUDA library.  Inputs are numpy arrays (or anything ``np.asarray`` takes); bf16
data must be widened exactly to float64 by the caller (see ``bf16_bits_to_f64``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bfq_oracle.c")
_LIB = os.path.join(_HERE, "libbfq_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no FMA contraction, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        i64, i32 = ctypes.c_int64, ctypes.c_int
        P = ctypes.c_void_p
        L.orc_forward.argtypes = [i64, P, P, i64, i64, P, i64]
        L.orc_inverse.argtypes = [i64, P, P, i64, i64, P, i64]
        L.orc_hadamard.argtypes = [i64, P, i64, i64, P, i64]
        L.orc_hadamard.restype = i32
        L.orc_dense_stage.argtypes = [i64, i32, P, P]
        L.orc_quantize.argtypes = [i64, i32, P, i64, i64, P, P, P, P]
        L.orc_pack.argtypes = [i64, i32, P, i64, P]
        L.orc_unpack.argtypes = [i64, i32, P, i64, P]
        L.orc_backward.argtypes = [i64, P, P, P, i64, i64, P, i64, P]
        L.orc_forward_quant.argtypes = [i64, P, P, i64, i64, i32, P, P, P]
        L.orc_f32_to_f16_sat.argtypes = [ctypes.c_float]
        L.orc_f32_to_f16_sat.restype = ctypes.c_uint16
        L.orc_f16_to_f64.argtypes = [ctypes.c_uint16]
        L.orc_f16_to_f64.restype = ctypes.c_double
        L.orc_num_threads.restype = i32
        for f in ("orc_forward", "orc_inverse", "orc_dense_stage", "orc_quantize", "orc_pack",
                  "orc_unpack", "orc_backward", "orc_forward_quant"):
            getattr(L, f).restype = i32
        _lib = L
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def bf16_bits_to_f64(bits) -> np.ndarray:
    """uint16/int16 bf16 bit patterns -> float64, exactly."""
    u = np.asarray(bits).view(np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)


def _theta(theta, n):
    th = _f64(theta)
    L = int(n).bit_length() - 1
    if th.shape != (L, n // 2):
        raise ValueError(f"theta must be [{L}][{n // 2}], got {th.shape}")
    return th


def forward(theta, x) -> np.ndarray:
    x = _f64(x)
    x2 = x.reshape(-1, x.shape[-1])
    n = x2.shape[1]
    th = _theta(theta, n)
    y = np.empty_like(x2)
    _check(lib().orc_forward(n, _ptr(th), _ptr(x2), x2.shape[0], n, _ptr(y), n), "forward")
    return y.reshape(x.shape)


def inverse(theta, y) -> np.ndarray:
    y = _f64(y)
    y2 = y.reshape(-1, y.shape[-1])
    n = y2.shape[1]
    th = _theta(theta, n)
    x = np.empty_like(y2)
    _check(lib().orc_inverse(n, _ptr(th), _ptr(y2), y2.shape[0], n, _ptr(x), n), "inverse")
    return x.reshape(y.shape)


def hadamard(x) -> np.ndarray:
    """y = H_n x per row, H_n the normalised Sylvester-Hadamard matrix of the paper's Sec. 3.1.1."""
    x = _f64(x)
    x2 = x.reshape(-1, x.shape[-1])
    n = x2.shape[1]
    y = np.empty_like(x2)
    _check(lib().orc_hadamard(n, _ptr(x2), x2.shape[0], n, _ptr(y), n), "hadamard")
    return y.reshape(x.shape)


def dense_stage(n: int, s: int, theta_s) -> np.ndarray:
    th = _f64(theta_s)
    assert th.shape == (n // 2,)
    M = np.empty((n, n), dtype=np.float64)
    _check(lib().orc_dense_stage(n, s, _ptr(th), _ptr(M)), "dense_stage")
    return M


def quantize(y, bits: int, scale_in=None, want_prequant: bool = False):
    """-> (codes int8 [rows][n], scale_f16 uint16 [rows][, prequant float64])."""
    y = _f64(y)
    y2 = y.reshape(-1, y.shape[-1])
    rows, n = y2.shape
    codes = np.empty((rows, n), dtype=np.int8)
    scales = np.empty(rows, dtype=np.uint16)
    sin = None
    if scale_in is not None:
        sin = np.ascontiguousarray(np.asarray(scale_in, dtype=np.uint16))
        assert sin.shape == (rows,)
    pre = np.empty((rows, n), dtype=np.float64) if want_prequant else None
    _check(lib().orc_quantize(n, bits, _ptr(y2), rows, n, _ptr(codes), _ptr(scales),
                              _ptr(sin) if sin is not None else None,
                              _ptr(pre) if pre is not None else None), "quantize")
    return (codes, scales, pre) if want_prequant else (codes, scales)


def pack(codes, bits: int) -> np.ndarray:
    c = np.ascontiguousarray(np.asarray(codes, dtype=np.int8))
    c2 = c.reshape(-1, c.shape[-1])
    rows, n = c2.shape
    out = np.empty((rows, n * bits // 8), dtype=np.uint8)
    _check(lib().orc_pack(n, bits, _ptr(c2), rows, _ptr(out)), "pack")
    return out


def unpack(packed, bits: int) -> np.ndarray:
    p = np.ascontiguousarray(np.asarray(packed, dtype=np.uint8))
    p2 = p.reshape(-1, p.shape[-1])
    rows, nb = p2.shape
    n = nb * 8 // bits
    out = np.empty((rows, n), dtype=np.int8)
    _check(lib().orc_unpack(n, bits, _ptr(p2), rows, _ptr(out)), "unpack")
    return out


def f16_bits_to_f64(bits) -> np.ndarray:
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def dequantize(codes, scale_f16) -> np.ndarray:
    """Dequant(q) = s * q with the stored fp16 scale (Sec. 3.4)."""
    return np.asarray(codes, dtype=np.float64) * f16_bits_to_f64(scale_f16)[:, None]


def code_histogram(codes, bits: int) -> np.ndarray:
    """Counts of every code value, index = code + 2^(bits-1) (the bins of the paper's P_bins, Sec. 3.4)."""
    c = np.asarray(codes, dtype=np.int64).reshape(-1) + (1 << (bits - 1))
    return np.bincount(c, minlength=1 << bits).astype(np.int64)


def uniformity_kl(hist) -> float:
    """L_uniform = D_KL(P_bins || U) = sum_i p_i log(p_i * number of bins), 0 log 0 = 0 (Sec. 3.4)."""
    h = np.asarray(hist, dtype=np.float64)
    p = h / h.sum()
    nz = p > 0
    return float(np.sum(p[nz] * np.log(p[nz] * h.size)))


def row_moments(y) -> np.ndarray:
    """[rows][2]: sum y^2 and sum y^4 per row, in float64."""
    y = _f64(y)
    y2 = y.reshape(-1, y.shape[-1])
    sq = y2 * y2
    return np.stack([sq.sum(axis=1), (sq * sq).sum(axis=1)], axis=1)


def cayley(params, n1: int) -> np.ndarray:
    """Q1 = (I - A)(I + A)^{-1}, A skew-symmetric with the n1 (n1 - 1) / 2 parameters in its upper triangle,
    row by row (paper Sec. 3.3, "Concrete Example for d = 5120")."""
    p = _f64(params).reshape(-1)
    if p.size != n1 * (n1 - 1) // 2:
        raise ValueError("need n1 (n1 - 1) / 2 parameters")
    A = np.zeros((n1, n1))
    A[np.triu_indices(n1, 1)] = p
    A = A - A.T
    I = np.eye(n1)
    return np.linalg.solve((I + A).T, (I - A).T).T  # X (I + A) = (I - A)


def composite_forward(Q1, theta2, x) -> np.ndarray:
    """y = (Q1 kron Q2) x per row, Q2 the butterfly of theta2 (Sec. 3.3): with x as an n1 x n2 matrix X,
    Y = Q1 (X Q2^T): Q2 on every run of n2 consecutive elements, then Q1 across the n1 runs."""
    Q1 = _f64(Q1)
    n1 = Q1.shape[0]
    x = _f64(x)
    rows = x.reshape(-1, x.shape[-1])
    n2 = rows.shape[1] // n1
    inner = forward(theta2, rows.reshape(-1, n2)).reshape(rows.shape[0], n1, n2)
    return np.einsum("ik,rkj->rij", Q1, inner).reshape(x.shape)


def composite_inverse(Q1, theta2, y) -> np.ndarray:
    """x = (Q1 kron Q2)^T y per row (= the inverse: both factors are orthogonal, Sec. 3.3): with y as an n1 x n2 matrix Y,
    X = (Q1^T Y) Q2: Q1^T across the n1 runs, then Q2^T = the inverse butterfly on every run."""
    Q1 = _f64(Q1)
    n1 = Q1.shape[0]
    y = _f64(y)
    rows = y.reshape(-1, y.shape[-1])
    n2 = rows.shape[1] // n1
    mixed = np.einsum("ki,rkj->rij", Q1, rows.reshape(rows.shape[0], n1, n2))
    return inverse(theta2, mixed.reshape(-1, n2)).reshape(y.shape)


def backward(theta, x, g):
    """-> (dx float64 [rows][n], dtheta float64 [L][n/2] summed over rows)."""
    x = _f64(x)
    g = _f64(g)
    x2 = x.reshape(-1, x.shape[-1])
    g2 = g.reshape(-1, g.shape[-1])
    assert x2.shape == g2.shape
    rows, n = x2.shape
    th = _theta(theta, n)
    dx = np.empty_like(x2)
    dth = np.empty_like(th)
    _check(lib().orc_backward(n, _ptr(th), _ptr(x2), _ptr(g2), rows, n, _ptr(dx), n, _ptr(dth)),
           "backward")
    return dx.reshape(x.shape), dth


def forward_quant(theta, x, bits: int, want_y: bool = False):
    """-> (packed uint8 [rows][n*bits/8], scale_f16 uint16 [rows][, y float64])."""
    x = _f64(x)
    x2 = x.reshape(-1, x.shape[-1])
    rows, n = x2.shape
    th = _theta(theta, n)
    packed = np.empty((rows, n * bits // 8), dtype=np.uint8)
    scales = np.empty(rows, dtype=np.uint16)
    y = np.empty((rows, n), dtype=np.float64) if want_y else None
    _check(lib().orc_forward_quant(n, _ptr(th), _ptr(x2), rows, n, bits, _ptr(packed),
                                   _ptr(scales), _ptr(y) if y is not None else None),
           "forward_quant")
    return (packed, scales, y) if want_y else (packed, scales)


def fold_weights(theta, W, bits: int, want_y: bool = False):
    """W Q^T row by row: row i of W Q^T is (Q w_i)^T, then per-row quantization."""
    return forward_quant(theta, W, bits, want_y)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def f32_to_f16_bits(v: float) -> int:
    return int(lib().orc_f32_to_f16_sat(ctypes.c_float(v)))


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
