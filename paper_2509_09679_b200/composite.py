"""Gradients of the composite transform Q = Q1 (x) Q2 (paper Sec. 3.3) composed from the library's entry points.

With a token row as an n1 x n2 matrix X and Y = Q1 (X Q2^T), for an upstream gradient G = dL/dY:

    G' = Q1^T G                       gradient at X' = X Q2^T (the rows after the butterfly)
    dL/dX      = G' Q2                = bfq_composite_inverse(G): per run, dx of the butterfly for upstream G'
    dL/dtheta2 = butterfly d-theta of the n1 * tokens runs with upstream G'   (bfq_backward on the n2-point plan)
    dL/dQ1     = sum over tokens of G X'^T                                    (a small dense product)
    dL/dparams = dL/dQ1 pulled back through Q1 = (I - A)(I + A)^-1 (A skew from the parameters): with
                 M = (I + A)^-1, dQ1 = -(I + Q1) dA M, so dL/dA = -(I + Q1)^T (dL/dQ1) M^T and the parameter (i < j)
                 receives dL/dA[i][j] - dL/dA[j][i].

Everything that touches the butterfly runs in the bfq kernels; the n1 x n1 algebra is torch in float64.
"""
from __future__ import annotations

import torch

from .binding import Plan


def cayley_pullback(params: torch.Tensor, n1: int, dQ1: torch.Tensor) -> torch.Tensor:
    """dL/dparams from dL/dQ1 (both on the same device; float64 inside)."""
    p = params.double()
    iu = torch.triu_indices(n1, n1, 1, device=p.device)
    A = torch.zeros((n1, n1), dtype=torch.float64, device=p.device)
    A[iu[0], iu[1]] = p
    A = A - A.t()
    eye = torch.eye(n1, dtype=torch.float64, device=p.device)
    M = torch.linalg.inv(eye + A)
    Q1 = (eye - A) @ M
    dA = -(eye + Q1).t() @ dQ1.double() @ M.t()
    return (dA - dA.t())[iu[0], iu[1]].to(params.dtype)


def composite_backward(plan: Plan, q1: torch.Tensor, params: torch.Tensor | None, x: torch.Tensor, g: torch.Tensor):
    """x, g: [tokens][n1 * n2] (same dtype).  Returns (dx, dtheta2, dQ1, dparams or None)."""
    n1, n2 = q1.shape[0], plan.n
    tokens = x.shape[0]
    gp = torch.einsum("ki,rkj->rij", q1, g.reshape(tokens, n1, n2).float())      # G' = Q1^T G
    runs_x = x.reshape(tokens * n1, n2)
    runs_g = gp.reshape(tokens * n1, n2).to(x.dtype)
    dx_runs, dtheta2 = plan.backward(runs_x, runs_g)                             # dx = G' Q2 per run, d-theta summed over runs
    xp = plan.forward(runs_x, out_dtype=torch.float32).reshape(tokens, n1, n2)   # X' = X Q2^T
    dQ1 = torch.einsum("rij,rkj->ik", g.reshape(tokens, n1, n2).float(), xp)
    dparams = cayley_pullback(params, n1, dQ1) if params is not None else None
    return dx_runs.reshape(tokens, n1 * n2), dtheta2, dQ1, dparams
