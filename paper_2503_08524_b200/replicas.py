"""Replica bookkeeping of the multi-GPU benchmark.

Sequences are independent and every replica holds the full weights, so N GPUs
run N copies of the step with no exchange on the data path.  What the ranks
share is only the measurement: the slowest replica's time bounds the job, and
the job's throughput is the units all replicas processed over that time.
"""
from __future__ import annotations

from typing import Optional

import torch


class Replicas:
    """Barrier, max-over-ranks time and whole-job throughput over an (optional)
    torch.distributed process group; with no group every call is the 1-rank case."""

    def __init__(self, dist=None, device: Optional[str] = None):
        self.dist = dist if (dist is not None and dist.is_initialized()) else None
        self.device = device or "cpu"
        self.world = self.dist.get_world_size() if self.dist else 1
        self.rank = self.dist.get_rank() if self.dist else 0

    def barrier(self) -> None:
        if self.dist is not None:
            self.dist.barrier()
        if str(self.device).startswith("cuda"):
            torch.cuda.synchronize()

    def max_ms(self, ms: float) -> float:
        """The slowest rank's time."""
        if self.dist is None:
            return float(ms)
        t = torch.tensor([ms], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def total_units(self, units: int) -> int:
        """Units (tokens) processed by all ranks together."""
        if self.dist is None:
            return int(units)
        t = torch.tensor([units], dtype=torch.int64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return int(t.item())

    def throughput(self, units_local: int, ms_local: float) -> float:
        """Whole-job units per second: all ranks' units over the slowest rank's time."""
        return self.total_units(units_local) / (self.max_ms(ms_local) / 1e3)
