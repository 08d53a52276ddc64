"""Token sharding of the layer across data-parallel ranks (one process per GPU).

The routed layer has no exchange step when tokens are split across ranks: every
rank plans and runs its own T tokens against a full copy of the expert weights.
What the ranks share is only bookkeeping, collected here so that it can be
exercised with the gloo backend on CPU: which batch a rank owns, the
max-over-ranks reduction of device times, and the whole-job throughput.
No layer arithmetic lives in this module.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist

from . import synth


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) as set by torch.distributed.run; (0, 0, 1) when launched plainly."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def rank_workload(base: synth.Workload, rank: int) -> synth.Workload:
    """The batch rank `rank` owns: same shapes and load recipe, its own random streams (rank 0 keeps the base seed)."""
    return synth.reseeded(base, base.seed + 1000 * rank) if rank else base


def max_over_ranks(value: float, device: torch.device, world: int) -> float:
    """Largest `value` over all ranks (every rank gets it); the job is as slow as its slowest rank."""
    if world <= 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def job_tokens_per_sec(world: int, tokens_per_rank: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank processed tokens_per_rank tokens in the (max-over-ranks) step time."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)
