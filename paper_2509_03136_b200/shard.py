"""Host-side plumbing for running the pass on several GPUs, one process per GPU.

The pass has no exchange step: Section 3.2 of the paper makes every computation per request and
per head, and layers are independent too.  Ranks therefore take disjoint requests (weak scaling)
and never read each other's memory.  What the ranks do share is bookkeeping: the job's time is the
slowest rank's, and an engine may want every rank's per-head budgets.  Both are tiny collectives
on `torch.distributed` (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from dataclasses import replace
from typing import List

import torch


def rank_workload(cfg, rank: int):
    """The workload of one rank: same shapes, its own requests (a seed of its own)."""
    return replace(cfg, seed=cfg.seed + 1000 * rank)


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The largest of the ranks' values (a job is as slow as its slowest rank)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_rank: int, world: int, seconds: float) -> float:
    """Whole-job cached tokens compressed per second when every rank handles `tokens_per_rank`."""
    return world * tokens_per_rank / seconds


def gather_budgets(budget: torch.Tensor, dist=None) -> List[torch.Tensor]:
    """Every rank's per-(request, KV head) budgets, in rank order (the one piece of the result an
    engine needs globally, to size its paged cache)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [budget]
    out = [torch.empty_like(budget) for _ in range(dist.get_world_size())]
    dist.all_gather(out, budget.contiguous())
    return out
