"""Multi-GPU plumbing for the benchmark: the path has no exchange step (tensor parallel 1
everywhere in the paper), so N GPUs run N independent replicas.  What crosses ranks is only the
barrier around the timed region and the maximum of the per-rank times.

Works with NCCL (one rank per GPU) and with gloo on CPU (tests)."""
from __future__ import annotations

import os
from typing import Optional

import torch


class Replicas:
    def __init__(self, backend: Optional[str] = None, device: Optional[torch.device] = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.device = device
        self._dist = None
        if self.world > 1:
            import torch.distributed as dist
            if backend is None:
                backend = "nccl" if (device is not None and device.type == "cuda") else "gloo"
            kwargs = {"device_id": device} if backend == "nccl" else {}
            dist.init_process_group(backend, **kwargs)
            self._dist = dist

    def barrier(self) -> None:
        if self._dist is not None:
            self._dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank's time: the job is as fast as its slowest replica."""
        if self._dist is None:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64,
                         device=self.device if (self.device is not None and self.device.type == "cuda") else "cpu")
        if t.is_cuda:
            t = t.float()
        self._dist.all_reduce(t, op=self._dist.ReduceOp.MAX)
        return float(t.item())

    def aggregate(self, units_per_rank: float, ms: float) -> float:
        """Whole-job throughput in units per second: every rank did `units_per_rank` in at most
        max-over-ranks `ms` milliseconds (weak scaling, independent replicas)."""
        return units_per_rank * self.world / (self.max_over_ranks(ms) * 1e-3)

    def close(self) -> None:
        if self._dist is not None:
            self._dist.destroy_process_group()
            self._dist = None
