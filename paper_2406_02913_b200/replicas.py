"""Rank plumbing of the multi-GPU benchmark: independent replicas, one process per GPU.

The ZO step holds the whole model on one GPU and exchanges nothing, so N GPUs run N replicas (weak
scaling).  What the ranks share is only the measurement: a barrier on both sides of the timed
region, the slowest rank's time, and the sum of the work done.  Works with any torch.distributed
backend ("nccl" on GPUs, "gloo" in the CPU tests); with one process it needs no process group.
"""
from __future__ import annotations

import os

import torch


class Replicas:
    def __init__(self, backend: str | None = None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"))
            self.dist = dist
        self.device = torch.device("cuda", self.local_rank) if (
            torch.cuda.is_available() and (backend or "nccl") == "nccl") else torch.device("cpu")

    def barrier(self) -> None:
        """Every rank's queued GPU work is done before and after the ranks meet."""
        if self.device.type == "cuda":
            torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        if self.device.type == "cuda":
            torch.cuda.synchronize()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank's time: what a job that waits for all replicas sees."""
        if self.dist is None:
            return float(value)
        t = torch.tensor([value], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, ms: float) -> float:
        """Units per second of all replicas together, from the max-over-ranks time in ms."""
        return self.world * units_per_rank * 1e3 / ms

    def close(self) -> None:
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None
