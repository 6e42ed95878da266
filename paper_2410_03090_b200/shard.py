"""Host-side helpers for running the pass on several GPUs.

Every unit (batch, layer, KV head) is independent in all stages except the budget rule, which couples only
the heads of one layer (or one sequence).  Whole sequences therefore shard across ranks with no collective
on the data path; ranks only agree on timing (barrier, maximum of the device-measured time)."""
from __future__ import annotations

from dataclasses import replace

import torch
import torch.distributed as dist

from .synth import Workload


def rank_workload(base: Workload, rank: int) -> Workload:
    """The shard of rank `rank`: its own sequence(s) of the same shape (weak scaling)."""
    return replace(base, seed=base.seed + 7919 * rank)


def max_over_ranks(value: float, device: torch.device | str, world: int) -> float:
    if world <= 1:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(wl: Workload, world: int, ms_per_step: float) -> float:
    """Tokens of all ranks per second, with the step time of the slowest rank."""
    return wl.B * wl.N * world / (ms_per_step / 1e3)
