"""Rank plumbing for runs on several GPUs of one node.  The path does not shard: rows are independent, there is no
exchange step, so N GPUs run N independent replicas (one process per GPU) and the only collectives are the barrier
around the timed region and the max over ranks of the measured time."""
from __future__ import annotations

import os

import torch


class Replicas:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE (as set by torch.distributed.run) and, for more than one rank, joins the
    process group (nccl when a CUDA device is given, gloo otherwise; MASTER_ADDR / MASTER_PORT from the environment)."""

    def __init__(self, device: torch.device | None = None, backend: str | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist

            backend = backend or ("nccl" if device is not None and device.type == "cuda" else "gloo")
            if backend == "nccl":
                dist.init_process_group(backend, device_id=device)
            else:
                dist.init_process_group(backend)
            self.dist = dist

    def seed(self, base: int) -> int:
        """Each replica draws its own rows."""
        return base + 100 * self.rank

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        if self.device is not None and self.device.type == "cuda":
            torch.cuda.synchronize(self.device)

    def max_over_ranks(self, v: float) -> float:
        if self.dist is None:
            return float(v)
        t = torch.tensor([v], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: int, ms: float) -> float:
        """Units all ranks processed per second, ms being the max over ranks of the time of one step."""
        return self.world * units_per_rank / (ms * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
