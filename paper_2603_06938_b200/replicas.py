"""Plumbing of multi-GPU runs.  The token mixer has no exchange step: sequences are independent,
so N GPUs run N independent replicas, each on its own batch, and nothing crosses the links on the
data path.  What the ranks share is only the measurement: a barrier around the timed region and
the maximum of the per-rank times.  Nothing here touches a GPU, so the same code runs under the
`gloo` backend in the CPU tests and under `nccl` in the benchmark.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch


def rank_env() -> Tuple[int, int, int]:
    """(rank, world size, local rank) as torchrun exports them; (0, 1, 0) for a plain launch."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(rank: int, index: int) -> int:
    """Seed of input set `index` of replica `rank`: every replica works on its own batch."""
    return 1000 * rank + index


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's figure (every rank gets it); the value itself without a process group."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(world: int, units_per_rank: int, ms_per_step: float) -> float:
    """Units per second of the whole job: all ranks' units over the slowest rank's step time."""
    return world * units_per_rank / (ms_per_step * 1e-3)
