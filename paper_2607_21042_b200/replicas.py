"""Multi-GPU = independent replicas.

Utterances are independent (the paper batches concurrent utterances, Section II-B) and the model is
1 GB, so several GPUs run several engines, each with the full weights and its own KV pool; the
decode path has no exchange step and uses no collective.  What is left for the host:

* ``StreamRouter``: which replica gets a new utterance (least reserved KV pages first).
* ``max_over_ranks`` / ``sum_over_ranks``: the only cross-rank traffic of ``bench.py --gpus N`` —
  the timing reduction (max of the per-rank device times) and the token count.  They go through
  ``torch.distributed`` and therefore work on any backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from dataclasses import dataclass, field

import torch
import torch.distributed as dist


def launch_ranks(script: str, argv, n_ranks: int, port: int = 0) -> int:
    """Runs `script argv...` as n_ranks processes of one node (one per GPU) under
    torch.distributed.run, rendezvous on 127.0.0.1, and returns its exit code.  Each rank finds
    RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in its environment."""
    if port <= 0:
        s = socket.socket()
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
        s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(int(n_ranks)),
           "--master-addr", "127.0.0.1", "--master-port", str(port), script] + list(argv)
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", "4")
    return subprocess.call(cmd, env=env)


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank scalar over the default process group (identity without one)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(tokens_this_rank: int, ms_this_rank: float, device=None) -> float:
    """tokens/s of the whole job: all ranks' tokens over the slowest rank's device time."""
    total = sum_over_ranks(tokens_this_rank, device)
    ms = max_over_ranks(ms_this_rank, device)
    return total / (ms * 1e-3)


@dataclass
class StreamRouter:
    """Assigns new utterances to replicas.  Each replica has `pages_per_replica` KV pages of 64
    tokens and `slots_per_replica` stream slots; an utterance reserves pages for its whole expected
    context up front (prefix + expected decode length) so that a replica never runs out mid-way."""
    n_replicas: int
    pages_per_replica: int
    slots_per_replica: int
    reserved: list = field(default_factory=list)      # pages reserved per replica
    open_streams: list = field(default_factory=list)  # {handle: pages} per replica
    _next: int = 0

    def __post_init__(self):
        self.reserved = [0] * self.n_replicas
        self.open_streams = [dict() for _ in range(self.n_replicas)]

    @staticmethod
    def pages_for(tokens: int) -> int:
        return (int(tokens) + 63) // 64

    def assign(self, expected_context: int):
        """Returns (replica, handle) or None if no replica can take the utterance now."""
        need = self.pages_for(expected_context)
        best = None
        for r in range(self.n_replicas):
            if len(self.open_streams[r]) >= self.slots_per_replica:
                continue
            if self.reserved[r] + need > self.pages_per_replica:
                continue
            if best is None or self.reserved[r] < self.reserved[best]:
                best = r
        if best is None:
            return None
        h = self._next
        self._next += 1
        self.open_streams[best][h] = need
        self.reserved[best] += need
        return best, h

    def release(self, replica: int, handle: int):
        need = self.open_streams[replica].pop(handle)
        self.reserved[replica] -= need
