"""Host-side plumbing for running the pass on several GPUs, one process per GPU.

The pass has no exchange step: Section 3.2 of the paper makes every computation per request and
per head, and layers are independent too.  Ranks therefore take disjoint requests (weak scaling)
and never read each other's memory.  What the ranks do share is bookkeeping: the job's time is the
slowest rank's, and an engine may want every rank's per-head budgets.  Both are tiny collectives
on `torch.distributed` (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import socket
import sys
from dataclasses import replace
from typing import List, Mapping, Optional, Sequence

import torch


def self_launch_command(script: str, argv: Sequence[str], n_gpus: int, env: Mapping[str, str],
                        port: Optional[int] = None) -> Optional[List[str]]:
    """The command that starts one rank per GPU for `script argv`, or None when nothing has to be started:
    a single GPU, or a launcher has already set up the ranks (WORLD_SIZE in the environment: its RANK /
    LOCAL_RANK / MASTER_* are used as they are).  The rendezvous is on 127.0.0.1 (one node)."""
    if n_gpus <= 1 or "WORLD_SIZE" in env:
        return None
    if port is None:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), script, *argv]


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
