"""Process-group plumbing for running independent replicas of the engine, one per GPU.

The event update never exchanges data between GPUs (every operation is element-wise over the
parameter dimension and the population lives on one device), so ranks only meet at a barrier
and at a max-reduction of their timings. `nccl` on GPUs, `gloo` in CPU tests."""
from __future__ import annotations

import os


class Ranks:
    def __init__(self, backend: str | None = None, device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist

            if not dist.is_initialized():
                os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
                os.environ.setdefault("MASTER_PORT", "29500")
                dist.init_process_group(backend=backend or "nccl", rank=self.rank, world_size=self.world)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def _tensor(self, values):
        import torch

        return torch.tensor(values, dtype=torch.float64, device=self.device if self.device is not None else "cpu")

    def max_over_ranks(self, value: float) -> float:
        if self.dist is None:
            return float(value)
        t = self._tensor([value])
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, value: float) -> float:
        if self.dist is None:
            return float(value)
        t = self._tensor([value])
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return float(t.item())

    def close(self):
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None


def aggregate_throughput(ranks: Ranks, units_this_rank: float, seconds_this_rank: float) -> tuple[float, float]:
    """Whole-job throughput of independent replicas: all ranks' units over the slowest rank's
    time. Returns (units per second, slowest time in seconds)."""
    slowest = ranks.max_over_ranks(seconds_this_rank)
    total = ranks.sum_over_ranks(units_this_rank)
    return total / slowest, slowest
