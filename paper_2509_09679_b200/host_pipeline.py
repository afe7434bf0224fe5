"""Forward + quantize for rows that live in (pinned) host memory, through the library's host-buffer entry point
(bfq_forward_quant_host): the rows are cut into chunks and the host -> device copy of one chunk, the kernels of another
and the device -> host copy of the codes of a third run at the same time, so that a call costs about as much as its
slowest leg (the host -> device copy) instead of the sum of the three.  This module only owns the device workspace."""
from __future__ import annotations

import torch

from .binding import Plan


class HostForwardQuant:
    """plan: a Plan whose angles the caller sets; rows / bits / dtype fix the workspace (two chunks of rows with their
    codes and scales).  call(x_host, codes_host, scales_host) with pinned host tensors returns after enqueueing on the
    current stream; the host buffers hold the results when that stream has drained."""

    def __init__(self, plan: Plan, rows: int, bits: int, dtype=torch.bfloat16, chunks: int = 8):
        self.plan, self.rows, self.bits = plan, int(rows), int(bits)
        chunk = max(8, -(-self.rows // max(1, chunks)))
        nbytes = plan.forward_quant_host_workspace(dtype, bits, chunk)
        self.workspace = torch.empty((nbytes,), dtype=torch.uint8, device=plan.device)

    def __call__(self, x_host: torch.Tensor, codes_host: torch.Tensor, scales_host: torch.Tensor, before=None):
        """before: optional callable run on the current stream ahead of the call (e.g. plan.set_angles)."""
        if before is not None:
            before()
        self.plan.forward_quant_host(x_host, self.bits, codes_host, scales_host, self.workspace)
