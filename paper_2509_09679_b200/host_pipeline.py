"""Forward + quantize for rows that live in (pinned) host memory: the rows are cut into chunks and the host -> device
copy of chunk c + 1, the kernels of chunk c and the device -> host copy of the codes of chunk c - 1 run on three
streams at the same time, so that a call costs about as much as its slowest leg (the host -> device copy) instead of the
sum of the three.  Everything that computes is a bfq call; this module only moves bytes and orders streams."""
from __future__ import annotations

import torch

from .binding import Plan


class HostForwardQuant:
    """plan: a Plan whose angles the caller sets; rows / bits / dtype fix the buffers.  call(x_host, codes_host,
    scales_host) with pinned host tensors; returns after enqueueing, `done` (a CUDA event on the caller's current
    stream) marks completion."""

    def __init__(self, plan: Plan, rows: int, bits: int, dtype=torch.bfloat16, chunks: int = 8):
        self.plan, self.rows, self.bits, self.n = plan, int(rows), int(bits), plan.n
        dev = plan.device
        self.chunk = max(1, -(-self.rows // max(1, chunks)))
        self.nchunks = -(-self.rows // self.chunk)
        self.x_dev = [torch.empty((self.chunk, self.n), dtype=dtype, device=dev) for _ in range(2)]
        self.codes_dev = torch.empty((self.rows, self.n * bits // 8), dtype=torch.uint8, device=dev)
        self.scales_dev = torch.empty((self.rows,), dtype=torch.float16, device=dev)
        self.s_in, self.s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        self.loaded = [torch.cuda.Event() for _ in range(2)]    # x_dev[b] holds its chunk
        self.consumed = [torch.cuda.Event() for _ in range(2)]  # the kernels have read x_dev[b]
        self.computed = torch.cuda.Event()

    def __call__(self, x_host: torch.Tensor, codes_host: torch.Tensor, scales_host: torch.Tensor, before=None):
        """before: optional callable run on the compute stream ahead of the first chunk (e.g. plan.set_angles)."""
        main = torch.cuda.current_stream(self.plan.device)
        self.s_in.wait_stream(main)
        self.s_out.wait_stream(main)
        if before is not None:
            before()
        for c in range(self.nchunks):
            b, r0 = c & 1, c * self.chunk
            r1 = min(self.rows, r0 + self.chunk)
            with torch.cuda.stream(self.s_in):
                if c >= 2:
                    self.s_in.wait_event(self.consumed[b])
                self.x_dev[b][: r1 - r0].copy_(x_host[r0:r1], non_blocking=True)
                self.loaded[b].record(self.s_in)
            main.wait_event(self.loaded[b])
            self.plan.forward_quant(self.x_dev[b][: r1 - r0], self.bits, codes=self.codes_dev[r0:r1],
                                    scales=self.scales_dev[r0:r1])
            self.consumed[b].record(main)
            self.computed.record(main)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(self.computed)
                codes_host[r0:r1].copy_(self.codes_dev[r0:r1], non_blocking=True)
                scales_host[r0:r1].copy_(self.scales_dev[r0:r1], non_blocking=True)
        main.wait_stream(self.s_out)
        main.wait_stream(self.s_in)
