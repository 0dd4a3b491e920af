"""One process per GPU, independent replicas: the only multi-process plumbing the emulation needs.

The emulated collective has no inter-GPU step (its ranks are buffers on one GPU), so N GPUs
run N replicas of the same workload.  What is shared is the timing protocol: a barrier on both
sides of the timed region and the slowest rank's device time.  Works over NCCL (one GPU per
rank) and over gloo (CPU, used by the tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


class Replicas:
    def __init__(self, backend: str | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
        self.cuda = self.backend == "nccl"
        if self.cuda:
            torch.cuda.set_device(self.local)
        if self.world > 1 and not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29511")
            kw = {"device_id": torch.device("cuda", self.local)} if self.cuda else {}
            dist.init_process_group(self.backend, rank=self.rank, world_size=self.world, **kw)

    def barrier(self) -> None:
        """All ranks have reached this point and (on GPUs) drained their device."""
        if self.world > 1:
            dist.barrier()
        if self.cuda:
            torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        """The slowest rank's value: a time measured on each rank's own device."""
        if self.world == 1:
            return float(x)
        t = torch.tensor([float(x)], dtype=torch.float64, device="cuda" if self.cuda else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, x: float) -> float:
        """Units of work done by the whole job (every replica does its own)."""
        if self.world == 1:
            return float(x)
        t = torch.tensor([float(x)], dtype=torch.float64, device="cuda" if self.cuda else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def close(self) -> None:
        if self.world > 1 and dist.is_initialized():
            dist.destroy_process_group()
