"""Comparison rules shared by the GPU parity tests (and by the smoke check).

fp32 outputs:   max |out - ref| <= 1e-5 * max|x|  per row.
bf16 outputs:   |out - ref| <= 2^-8 |ref| + 1e-5 * max|x|   (one bf16 rounding on top).
codes / scales: the fp16 scale equals the oracle's or differs by exactly one fp16 ulp (the
                row absmax computed in fp32 may land on the other side of an fp16 rounding
                boundary); for such rows the oracle re-quantises with the GPU's scale.  Codes
                are then bit-exact except for off-by-one codes where the oracle's pre-rounding
                value lies within 1e-4 of a rounding boundary, at most 1e-4 of all elements.
                An exact tie (pre-rounding value exactly k + 1/2, which happens in bulk only for
                degenerate inputs such as theta = 0 on bf16 rows) has two nearest integers and the
                paper's round() names no tie rule: either neighbour is accepted and such elements
                do not count against the 1e-4 budget.
d-theta:        per stage  max_j |d - ref| <= 1e-4 * max_j |ref[s]|,  and  |d - ref|_2 <= 1e-4 |ref|_2.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def check_rows_close(out: torch.Tensor, ref: np.ndarray, x_absmax: np.ndarray, what: str = ""):
    o = to_f64(out)
    assert o.shape == ref.shape, (o.shape, ref.shape)
    assert np.isfinite(o).all(), f"{what}: non-finite output"
    tol = 1e-5 * x_absmax.reshape(-1, 1)
    if out.dtype == torch.bfloat16:
        tol = tol + 2.0 ** -8 * np.abs(ref)
    err = np.abs(o - ref)
    bad = err > tol
    if bad.any():
        k = np.unravel_index(np.argmax(err - tol), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} elements out of tolerance; worst at {k}: "
                             f"err {err[k]:.3e} tol {np.broadcast_to(tol, err.shape)[k]:.3e}")
    return float((err / np.broadcast_to(tol, err.shape)).max())


def check_quant(codes_packed: torch.Tensor, scales: torch.Tensor, y_ref: np.ndarray, bits: int, what: str = ""):
    """y_ref: the oracle's fp64 rotated rows.  Returns a dict of counts for reporting."""
    rows, n = y_ref.shape
    got_codes = oracle.unpack(codes_packed.detach().cpu().numpy(), bits)
    got_s = scales.detach().cpu().view(torch.int16).numpy().view(np.uint16)
    ref_codes, ref_s, pre = oracle.quantize(y_ref, bits, want_prequant=True)
    ds = got_s.astype(np.int64) - ref_s.astype(np.int64)
    assert np.all(np.abs(ds) <= 1), f"{what}: fp16 scale off by more than one ulp in {np.sum(np.abs(ds) > 1)} rows"
    shifted = np.nonzero(ds != 0)[0]
    if shifted.size:
        c2, _, p2 = oracle.quantize(y_ref[shifted], bits, scale_in=got_s[shifted], want_prequant=True)
        ref_codes[shifted] = c2
        pre[shifted] = p2
    diff = got_codes.astype(np.int32) - ref_codes.astype(np.int32)
    bad = diff != 0
    nbad = int(bad.sum())
    if nbad:
        assert np.all(np.abs(diff[bad]) == 1), f"{what}: codes differ by more than one"
        frac = pre[bad] - np.floor(pre[bad])
        dist = np.abs(frac - 0.5)
        assert np.all(dist < 1e-4), f"{what}: code mismatch away from a rounding boundary (dist {dist.max():.3e})"
        exact_tie = dist < 1e-12
        near = int(nbad - exact_tie.sum())
        assert near <= max(1, int(1e-4 * rows * n)), f"{what}: {near} boundary mismatches of {rows * n}"
    return {"rows": rows, "scale_ulp_rows": int(shifted.size), "boundary_codes": nbad}


def check_dtheta(dth: torch.Tensor, ref: np.ndarray, what: str = ""):
    d = to_f64(dth)
    assert d.shape == ref.shape
    assert np.isfinite(d).all()
    per_stage = np.abs(d - ref).max(axis=1) / np.maximum(np.abs(ref).max(axis=1), 1e-300)
    assert per_stage.max() <= 1e-4, f"{what}: per-stage relative error {per_stage}"
    rel = np.linalg.norm(d - ref) / max(np.linalg.norm(ref), 1e-300)
    assert rel <= 1e-4, f"{what}: global relative error {rel:.3e}"
    return float(per_stage.max()), float(rel)


class Guarded:
    """A device buffer with canary bytes either side, to catch out-of-bounds writes."""

    PAD = 4096

    def __init__(self, shape, dtype, device):
        numel = int(np.prod(shape)) if len(shape) else 1
        esz = torch.empty(0, dtype=dtype).element_size()
        self.nbytes = numel * esz
        total = self.nbytes + 2 * self.PAD
        self.raw = torch.full((total,), 0xA5, dtype=torch.uint8, device=device)
        self.view = self.raw[self.PAD:self.PAD + self.nbytes].view(dtype).view(*shape)

    def intact(self) -> bool:
        head = self.raw[:self.PAD]
        tail = self.raw[self.PAD + self.nbytes:]
        return bool((head == 0xA5).all().item() and (tail == 0xA5).all().item())
