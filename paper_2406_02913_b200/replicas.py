"""Rank plumbing for several GPUs, one process per GPU.

Two uses.  (1) Independent replicas (the benchmark's default): the ZO step holds the whole model on one
GPU and exchanges nothing; the ranks share only the measurement: a barrier on both sides of the timed
region, the slowest rank's time, and the sum of the work done.  (2) Data-parallel replicas of ONE
fine-tuning run: every rank holds the same weights, mask and S and uses the same (seed, step), so all
draw the same z; each evaluates f+ and f- on its own share of the batch (Definition 1's loss is a batch
mean), the ranks add up (sum of losses of f+, of f-, number of positions) -- 24 bytes per step -- and
every rank applies the identical update.  The sum is a torch.distributed all-reduce (NCCL on GPUs: the
remote values arrive in local memory; no kernel of the library reads a peer's memory).
Works with any backend ("nccl" on GPUs, "gloo" in the CPU tests); one process needs no process group.
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

    def sum_over_ranks(self, t: torch.Tensor) -> torch.Tensor:
        """In-place sum of a tensor over all ranks (the one exchange of a data-parallel ZO step)."""
        if self.dist is not None:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return t

    def data_parallel_step(self, losses_fn, apply_fn):
        """One ZO step of data-parallel replicas: losses_fn() -> fp64 tensor (sum f+, sum f-, count) of
        this rank's share of the batch (z drawn from the common (seed, step)); the sums are added over
        the ranks; apply_fn(sums) forms f+-, g and the update, identically on every rank."""
        return apply_fn(self.sum_over_ranks(losses_fn()))

    def whole_job_rate(self, units_per_rank: float, ms: float) -> float:
        """Units per second of all replicas together, from the max-over-ranks time in ms."""
        return self.world * units_per_rank * 1e3 / ms

    def close(self) -> None:
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None
