"""Multi-GPU plumbing of the benchmark: N independent replicas of the layer, one process per GPU.

The Switch FFN layer on one device has no exchange step (no all-to-all is built), so several GPUs only ever run
replicas: each rank routes and processes its own batch.  The only cross-rank traffic is measurement plumbing:
a barrier before and after the timed region and the maximum of the per-rank elapsed times.  The same code runs
with the `gloo` backend on CPU (that is how it is tested) and with `nccl` on GPUs.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


class Replicas:
    """Rank bookkeeping read from the torchrun environment (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_*)."""

    def __init__(self, backend: str | None = None, device: torch.device | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self._own_group = False
        if self.world > 1 and not dist.is_initialized():
            backend = backend or ("nccl" if device is not None and device.type == "cuda" else "gloo")
            kwargs = {"device_id": device} if backend == "nccl" and device is not None else {}
            dist.init_process_group(backend, **kwargs)
            self._own_group = True

    def barrier(self) -> None:
        if self.world > 1:
            dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank's value (every multi-GPU time is reported as the maximum over ranks)."""
        if self.world == 1:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def tokens_per_second(self, tokens_per_rank: int, ms_per_step: float) -> float:
        """Whole-job throughput of `world` replicas that each process tokens_per_rank tokens per step."""
        return self.world * tokens_per_rank / (ms_per_step * 1e-3)

    @property
    def is_reporting_rank(self) -> bool:
        return self.rank == 0

    def close(self) -> None:
        if self._own_group and dist.is_initialized():
            dist.barrier()
            dist.destroy_process_group()
