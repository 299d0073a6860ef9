"""Replica bookkeeping for runs on several GPUs.

The path has no exchange step (every (request, KV head) is independent), so N GPUs run N independent
replicas, each with its own host store share and host link. The only cross-rank work is the barrier
around the timed region and the aggregation below: the job's time is the slowest rank's, the job's
tokens are the sum over ranks. Works on any torch.distributed backend (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def aggregate(ms_local: float, tokens_local: int, device="cpu") -> tuple[float, int]:
    """Returns (max over ranks of the elapsed milliseconds, sum over ranks of the tokens processed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), int(tokens_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    n = torch.tensor([int(tokens_local)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def throughput(ms_local: float, tokens_local: int, device="cpu") -> float:
    """Whole-job tokens per second."""
    ms, n = aggregate(ms_local, tokens_local, device)
    return n / (ms * 1e-3)


def host_budget_per_rank(available_bytes: int, local_world: int, fraction: float = 0.6) -> int:
    """Pinned host memory one rank may use for its store share."""
    return int(available_bytes * fraction / max(1, local_world))


def gather_per_rank(value: float) -> list[float]:
    """The same scalar from every rank, in rank order (on every rank); [value] without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(value)]
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, float(value))
    return [float(v) for v in out]
