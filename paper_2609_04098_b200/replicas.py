"""Multi-GPU plumbing for the benchmark: the path has no exchange step (tensor parallel 1
everywhere in the paper), so N GPUs run N independent replicas.  What crosses ranks is only the
barrier around the timed region and the maximum of the per-rank times.

Works with NCCL (one rank per GPU) and with gloo on CPU (tests)."""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Optional, Sequence

import torch


def launched_by_a_launcher() -> bool:
    """True when RANK / WORLD_SIZE were exported by whoever started this process (torchrun or
    spawn_replicas): the process is then one replica and must not start more."""
    return "RANK" in os.environ and "WORLD_SIZE" in os.environ


def spawn_replicas(n: int, argv: Sequence[str], extra_env: Optional[dict] = None, timeout: Optional[float] = None) -> int:
    """Start `n` copies of `argv` on this node, one per GPU (RANK = LOCAL_RANK = 0..n-1, WORLD_SIZE = n,
    rendezvous on 127.0.0.1 at a free port), wait for all of them and return the first non-zero exit
    code (0 if all succeeded).  Rank 0 inherits this process's stdout, so the one line it prints is
    the job's output; the other ranks' stdout is discarded, every rank's stderr is inherited."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs: List[subprocess.Popen] = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        if extra_env:
            env.update(extra_env)
        procs.append(subprocess.Popen(list(argv), env=env, stdout=None if rank == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        try:
            code = p.wait(timeout=timeout)
        except subprocess.TimeoutExpired:
            p.kill()
            code = 124
        if code != 0 and rc == 0:
            rc = code
    return rc


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
