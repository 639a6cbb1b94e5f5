"""Replica bookkeeping for runs on more than one GPU.

The collectives keep all P simulated ranks in one GPU's memory and exchange
nothing between GPUs, so N GPUs run N independent replicas of the workload.
What the processes do share is the protocol of a measurement: a barrier on
both sides of the timed region, the slowest replica's time, and the sum of the
work done.  ``torch.distributed`` carries that (NCCL on GPUs, gloo on CPU for
the tests); no data-path collective exists.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank_world() -> tuple[int, int, int]:
    """(rank, world size, local rank) as torchrun exports them; (0, 1, 0) without torchrun."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


class Replicas:
    def __init__(self, backend: str | None = None, device: torch.device | None = None):
        self.rank, self.world, self.local_rank = env_rank_world()
        self.device = device if device is not None else torch.device("cpu")
        self.active = self.world > 1
        if self.active and not dist.is_initialized():
            backend = backend or ("nccl" if self.device.type == "cuda" else "gloo")
            kw = {"device_id": self.device} if backend == "nccl" else {}
            dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kw)

    def barrier(self) -> None:
        """All replicas reach this point; on a GPU also waits for the device."""
        if self.active:
            dist.barrier()
        if self.device.type == "cuda":
            torch.cuda.synchronize(self.device)

    def max(self, x: float) -> float:
        if not self.active:
            return float(x)
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum(self, x: float) -> float:
        if not self.active:
            return float(x)
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def whole_job_rate(self, units_this_replica: float, ms_this_replica: float) -> tuple[float, float]:
        """(units of all replicas per second, slowest replica's milliseconds)."""
        ms = self.max(ms_this_replica)
        units = self.sum(units_this_replica)
        return units / (ms * 1e-3), ms

    def close(self) -> None:
        if self.active and dist.is_initialized():
            dist.barrier()
            dist.destroy_process_group()
