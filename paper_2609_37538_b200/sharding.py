"""Multi-GPU host logic: tables (requests) are independent, so they shard over ranks with no data-path
collective.  Each rank runs its own context on its own GPU and host link; the only communication is the
reduction of counters and timings for reporting (max over ranks for device time, sum for work)."""
from __future__ import annotations

from typing import Dict, List, Sequence


def tables_of_rank(num_tables: int, world_size: int, rank: int) -> List[int]:
    """Contiguous, balanced split: the first num_tables % world_size ranks take one table more."""
    if world_size < 1 or not 0 <= rank < world_size:
        raise ValueError("bad rank %d of %d" % (rank, world_size))
    q, r = divmod(num_tables, world_size)
    begin = rank * q + min(rank, r)
    return list(range(begin, begin + q + (1 if rank < r else 0)))


def aggregate(times_ms: Dict[str, float], work: Dict[str, float], group=None):
    """Reduces per-rank device times (MAX) and work counters (SUM) over the process group.
    Works with any torch.distributed backend; tensors live on the CPU for gloo and on the current
    CUDA device for nccl.  Returns (times, work) dictionaries with the reduced values on every rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return dict(times_ms), dict(work)
    device = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    tk, wk = sorted(times_ms), sorted(work)
    t = torch.tensor([float(times_ms[k]) for k in tk], dtype=torch.float64, device=device)
    w = torch.tensor([float(work[k]) for k in wk], dtype=torch.float64, device=device)
    if tk:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    if wk:
        dist.all_reduce(w, op=dist.ReduceOp.SUM, group=group)
    return dict(zip(tk, t.tolist())), dict(zip(wk, w.tolist()))


def whole_job_gbs(bytes_all_ranks: float, max_time_ms: float) -> float:
    """Whole-job throughput: the bytes all ranks moved divided by the slowest rank's device time."""
    return bytes_all_ranks / 1e9 / (max_time_ms / 1e3)
