"""Host-side plumbing for running the verification step on several GPUs.

Sequences are independent problems (Section 3.4 verifies each sequence's own
tree against its own cache), so N ranks run N replicas of the step on N
different batches.  There is no exchange on the data path; `torch.distributed`
serves the barrier around the timed region and the max-over-ranks of the
device times only.  Everything here is backend-agnostic (NCCL on GPUs, gloo in
the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Sequence

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class RankInfo:
    rank: int
    local_rank: int
    world: int


def rank_info() -> RankInfo:
    """Rank, local rank and world size from the launcher's environment (1 process = 1 GPU)."""
    return RankInfo(int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
                    int(os.environ.get("WORLD_SIZE", "1")))


def shard_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch that `rank` verifies: every rank gets its own sequences."""
    return int(base_seed) + int(rank)


def max_over_ranks(values: Sequence[float], device: torch.device | str = "cpu") -> list[float]:
    """Element-wise maximum of `values` over all ranks (the values themselves when not distributed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def all_ok(ok: bool, device: torch.device | str = "cpu") -> bool:
    """True when every rank reports `ok` (a rank whose status words were set fails the whole job)."""
    return max_over_ranks([0.0 if ok else 1.0], device)[0] == 0.0


def whole_job_rate(units_per_rank: float, world: int, slowest_ms: float) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank` within `slowest_ms`."""
    if slowest_ms <= 0.0:
        raise ValueError("non-positive duration")
    return world * units_per_rank * 1e3 / slowest_ms
