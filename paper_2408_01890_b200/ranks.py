"""One process per GPU: the host-side plumbing of a multi-rank run.

The attention path shards over the batch with no exchange (independent sequences; the aligner mixes heads, so it does
not shard over heads): every rank runs the same step on its own sequences, and the only communication is the barrier
around the timed region and the maximum of the ranks' times.  `RankGroup` wraps exactly that; the backend is NCCL on
GPUs and gloo in the CPU tests.
"""
from __future__ import annotations

import os
from typing import Optional

import torch


class RankGroup:
    """Rank, world size and the two collectives a weak-scaling measurement needs."""

    def __init__(self, backend: Optional[str] = None, device: Optional[torch.device] = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device if device is not None else torch.device("cpu")
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            backend = backend or ("nccl" if self.device.type == "cuda" else "gloo")
            kwargs = {"device_id": self.device} if backend == "nccl" else {}
            dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kwargs)
            self.dist = dist

    def barrier(self) -> None:
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, x: float) -> float:
        """The slowest rank's time: what a whole-job throughput has to be divided by."""
        if self.dist is None:
            return float(x)
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def seed(self) -> int:
        """Every rank draws its own sequences: the synthetic input streams are keyed by this."""
        return self.rank

    def whole_job_per_second(self, units_per_rank: float, ms: float) -> float:
        """Weak scaling: every rank processed `units_per_rank`; `ms` is the maximum over the ranks."""
        return self.world * units_per_rank / (ms * 1e-3)

    def close(self) -> None:
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
