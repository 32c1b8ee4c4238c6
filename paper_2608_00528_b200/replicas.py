"""Host-side plumbing for running the decode path on several GPUs.

Sequences are independent (every (sequence, layer) is its own unit of Eq. 3-18), so the path shards by
sequence with no exchange step: each rank owns a batch of its own sequences and runs the single-GPU library on
it.  Nothing here touches the data path; the only communication is the reduction of the timing (max over
ranks) that the benchmark reports.  Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU
tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Replica:
    rank: int
    local_rank: int
    world: int

    @property
    def is_reporter(self) -> bool:
        return self.rank == 0


def replica_from_env(env=None) -> Replica:
    """Rank layout as torchrun exports it; a plain `python` launch is world size 1."""
    env = os.environ if env is None else env
    return Replica(int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0")), int(env.get("WORLD_SIZE", "1")))


def sequence_ids(rep: Replica, batch_per_rank: int) -> list[int]:
    """Global ids of the sequences this rank owns: rank-major, disjoint, covering [0, world * batch_per_rank)."""
    if batch_per_rank < 0 or not (0 <= rep.rank < rep.world):
        raise ValueError("bad replica layout")
    return list(range(rep.rank * batch_per_rank, (rep.rank + 1) * batch_per_rank))


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Slowest rank's figure (the time every whole-job rate is computed from); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(steps_per_rank: int, world: int, seconds: float) -> float:
    """Steps per second of the whole job: every rank ran `steps_per_rank` steps on its own batch (weak scaling)
    within `seconds`, the maximum over ranks."""
    if seconds <= 0:
        raise ValueError("non-positive duration")
    return world * steps_per_rank / seconds
