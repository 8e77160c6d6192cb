"""Replica plumbing for multi-GPU runs.

The pQuant linear layer has no exchange step (token rows are independent, weights are
replicated), so N GPUs run N independent replicas: one process per GPU, no collective on the
data path.  What the ranks share is bookkeeping only: a barrier around the timed region, the
maximum of the per-rank times, and the whole-job throughput computed from it.  The same code
runs over NCCL on GPUs and over gloo on CPUs (tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass
class Replicas:
    rank: int
    local_rank: int
    world: int
    backend: str | None = None

    @property
    def is_root(self) -> bool:
        return self.rank == 0

    def barrier(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max_over_ranks(self, value: float, device=None) -> float:
        """Largest `value` of any rank: a multi-GPU time is the slowest replica's."""
        if self.world == 1:
            return float(value)
        import torch
        import torch.distributed as dist
        t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, ms: float) -> float:
        """Units per second over all replicas, each of which processed `units_per_rank` in `ms` (the maximum over ranks)."""
        return self.world * units_per_rank / (ms * 1e-3)

    def close(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


def from_env(backend: str, device=None) -> Replicas:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE (as set by torch.distributed.run) and joins the process group when WORLD_SIZE > 1."""
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    return Replicas(rank, local, world, backend if world > 1 else None)
