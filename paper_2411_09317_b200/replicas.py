"""Multi-GPU plumbing for the replicas-only scaling mode: the path has no exchange step (sequences and slots are
independent units, the paper is single-GPU), so N GPUs run N independent replicas and only the *timing* is
combined: barrier before and after, maximum over ranks of the device-measured time, sum of the work.

Backend "nccl" on GPUs (bench.py), "gloo" on CPU (tests).  One process per GPU, launched by torch.distributed.run.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


class Replicas:
    def __init__(self, backend: str | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
        self.device = torch.device("cuda", self.local_rank) if self.backend == "nccl" else torch.device("cpu")
        if self.world > 1 and not dist.is_initialized():
            if self.backend == "nccl":
                torch.cuda.set_device(self.local_rank)
                dist.init_process_group("nccl", device_id=self.device)
            else:
                dist.init_process_group("gloo")

    def barrier(self) -> None:
        if self.world > 1:
            dist.barrier()
        if self.backend == "nccl":
            torch.cuda.synchronize()

    def _reduce(self, x: float, op) -> float:
        if self.world == 1:
            return float(x)
        t = torch.tensor([float(x)], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=op)
        return float(t.item())

    def max_over_ranks(self, x: float) -> float:
        return self._reduce(x, dist.ReduceOp.MAX)

    def sum_over_ranks(self, x: float) -> float:
        return self._reduce(x, dist.ReduceOp.SUM)

    def aggregate_throughput(self, units_this_rank: float, ms_this_rank: float) -> tuple[float, float]:
        """-> (units of all ranks / slowest rank's time in seconds, that time in ms)"""
        ms = self.max_over_ranks(ms_this_rank)
        units = self.sum_over_ranks(units_this_rank)
        return units / (ms * 1e-3), ms

    def close(self) -> None:
        if self.world > 1 and dist.is_initialized():
            dist.destroy_process_group()
