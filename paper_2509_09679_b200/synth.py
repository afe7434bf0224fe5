"""Seeded synthetic inputs for the butterfly-rotation path.

This module only draws numbers: angles, activation rows, weight rows and upstream
gradients, shaped like the workloads the paper describes (LLaMA hidden sizes 4096 /
8192, 128 x 2048-token calibration batches, heavy-tailed activations with a few
massive outlier channels).  It holds none of the method's arithmetic and is the one
module both the CPU oracle's tests and the CUDA path's tests/bench draw inputs from.

Every generator takes a ``device``: the same seed gives the same numbers on the same
device type (torch's CPU and CUDA generators are different streams).  A tensor made
on the GPU is the datum; rows handed to the CPU oracle are copied from it bit for bit.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch


def log2_exact(n: int) -> int:
    L = int(n).bit_length() - 1
    if n < 2 or (1 << L) != n:
        raise ValueError(f"n must be a power of two >= 2, got {n}")
    return L


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def angles(n: int, kind: str, seed: int, device="cpu") -> torch.Tensor:
    """theta[log2 n][n/2] fp32.  kind: 'uniform' = U[-pi, pi); 'normal' = N(pi/4, 0.3);
    'zero'; 'hadamard' = all pi/4."""
    L = log2_exact(n)
    shape = (L, n // 2)
    if kind == "zero":
        return torch.zeros(shape, dtype=torch.float32, device=device)
    if kind == "hadamard":
        return torch.full(shape, math.pi / 4, dtype=torch.float32, device=device)
    g = _gen(seed, device)
    if kind == "uniform":
        u = torch.rand(shape, generator=g, dtype=torch.float64, device=device)
        return ((u * 2.0 - 1.0) * math.pi).to(torch.float32)
    if kind == "normal":
        z = torch.randn(shape, generator=g, dtype=torch.float32, device=device)
        return (z * 0.3 + math.pi / 4).to(torch.float32)
    raise ValueError(kind)


def outlier_channels(n: int, k: int, seed: int) -> torch.Tensor:
    """First k entries of a seeded permutation of 0..n-1 (always drawn on the CPU so
    that the channel set does not depend on where the rows are generated)."""
    if k == 0:
        return torch.zeros(0, dtype=torch.int64)
    return torch.randperm(n, generator=_gen(seed ^ 0x5EED, "cpu"))[:k].clone()


def rows(
    n_rows: int,
    n: int,
    dist: str,
    seed: int,
    *,
    outliers: int = 0,
    outlier_scale: float = 1.0,
    scale: float = 1.0,
    dtype=torch.float32,
    device="cpu",
    chunk_rows: int = 8192,
) -> torch.Tensor:
    """[n_rows][n] values.  dist: 'normal' N(0,1); 'student_t3' = Z / sqrt(chi2_3 / 3);
    'laplace' Laplace(0,1) by inverse CDF.  ``outliers`` fixed channels are multiplied
    by ``outlier_scale``.  Generated in row chunks (chunk c uses seed + 7919*c) so the
    transient fp32 working set stays small at full size."""
    out = torch.empty((n_rows, n), dtype=dtype, device=device)
    ch = outlier_channels(n, outliers, seed).to(device)
    for c, r0 in enumerate(range(0, n_rows, chunk_rows)):
        r1 = min(n_rows, r0 + chunk_rows)
        g = _gen(seed + 7919 * c, device)
        shape = (r1 - r0, n)
        if dist == "normal":
            v = torch.randn(shape, generator=g, dtype=torch.float32, device=device)
        elif dist == "student_t3":
            z = torch.randn(shape, generator=g, dtype=torch.float32, device=device)
            chi = torch.zeros(shape, dtype=torch.float32, device=device)
            for _ in range(3):
                w = torch.randn(shape, generator=g, dtype=torch.float32, device=device)
                chi.addcmul_(w, w)
            v = z / torch.sqrt(chi / 3.0).clamp_min_(1e-6)
        elif dist == "laplace":
            u = torch.rand(shape, generator=g, dtype=torch.float32, device=device) - 0.5
            v = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp_max_(0.5 - 1e-7))
        else:
            raise ValueError(dist)
        if scale != 1.0:
            v *= scale
        if outliers:
            v[:, ch] *= outlier_scale
        out[r0:r1] = v.to(dtype)
    return out


def cayley_params(n1: int, seed: int, std: float = 0.1, device="cpu") -> torch.Tensor:
    """n1 (n1 - 1) / 2 entries N(0, std^2) for the strict upper triangle of a skew-symmetric matrix, row by row
    (the dense factor of the composite transform; a small std keeps the factor near the identity, as a learned
    factor initialised at identity would be)."""
    return std * torch.randn(n1 * (n1 - 1) // 2, generator=_gen(seed ^ 0xCA71E7, device), dtype=torch.float32, device=device)


# the composite example of the paper: hidden size 5120 = 40 x 128 (a LLaMA-13B-shaped activation row)
COMPOSITE_5120 = dict(n1=40, n2=128, n_rows=32768, dist="student_t3", outliers=8, outlier_scale=50.0, seed=6000)


@dataclass(frozen=True)
class Workload:
    """One of the named configurations (shapes and distributions only)."""

    name: str
    n: int
    n_rows: int
    dtype: torch.dtype
    dist: str
    outliers: int
    outlier_scale: float
    angle_kind: str
    bits: int
    scale: float = 1.0

    @property
    def L(self) -> int:
        return log2_exact(self.n)

    def theta(self, device="cpu", seed=None) -> torch.Tensor:
        return angles(self.n, self.angle_kind, self.seed if seed is None else seed, device)

    @property
    def seed(self) -> int:
        return 1000 * (1 + list(WORKLOADS).index(self.name))

    def x(self, device="cpu", n_rows=None, seed=None, dtype=None) -> torch.Tensor:
        return rows(
            self.n_rows if n_rows is None else n_rows,
            self.n,
            self.dist,
            (self.seed if seed is None else seed) + 1,
            outliers=self.outliers,
            outlier_scale=self.outlier_scale,
            scale=self.scale,
            dtype=self.dtype if dtype is None else dtype,
            device=device,
        )

    def g(self, device="cpu", n_rows=None, seed=None, dtype=None) -> torch.Tensor:
        """Upstream gradient dL/dy ~ N(0,1)."""
        return rows(
            self.n_rows if n_rows is None else n_rows,
            self.n,
            "normal",
            (self.seed if seed is None else seed) + 2,
            dtype=self.dtype if dtype is None else dtype,
            device=device,
        )


WORKLOADS = {
    # tiny correctness case: fp32 rows, angles uniform in [-pi, pi)
    "tiny256": Workload("tiny256", 256, 1024, torch.float32, "normal", 4, 20.0, "uniform", 4),
    # LLaMA-7B-shaped activation rotation + INT4 (the headline)
    "act4096_int4": Workload("act4096_int4", 4096, 32768, torch.bfloat16, "student_t3", 8, 50.0, "normal", 4),
    # angle-learning step: forward + backward on 128 x 2048 token rows
    "learn4096": Workload("learn4096", 4096, 262144, torch.bfloat16, "student_t3", 8, 50.0, "normal", 4),
    # LLaMA-70B-shaped 2-bit path
    "act8192_int2": Workload("act8192_int2", 8192, 65536, torch.bfloat16, "laplace", 16, 100.0, "normal", 2),
    # weight folding W Q^T, W 28672 x 8192, entries N(0, 0.02^2)
    "fold8192_int2": Workload("fold8192_int2", 8192, 28672, torch.bfloat16, "normal", 0, 1.0, "normal", 2, 0.02),
}


def checksum64(t: torch.Tensor) -> int:
    """Order-dependent 64-bit checksum of a tensor's raw bytes (for bench records)."""
    b = t.detach().contiguous().view(torch.uint8).reshape(-1).to("cpu")
    pad = (-b.numel()) % 8
    if pad:
        b = torch.cat([b, torch.zeros(pad, dtype=torch.uint8)])
    w = b.view(torch.int64)
    idx = torch.arange(1, w.numel() + 1, dtype=torch.int64)
    # wrapping int64 arithmetic
    return int(((w * (idx * 2 + 1)).sum().item()) & 0xFFFFFFFFFFFFFFFF)
