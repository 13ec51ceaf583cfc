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


# ---- placement on a multi-socket host ------------------------------------------------------------------------------
# Each rank's pinned host KV should sit in the memory of the socket its GPU hangs off, and the threads that fill
# it should run there (first touch decides the pages' NUMA node): rows read across the inter-socket link do not
# reach the GPU's full host-link rate.  Everything here only READS sysfs; no GPU or system setting is changed.

def pci_address(domain: int, bus: int, device: int, function: int = 0) -> str:
    """The sysfs name of a PCI function, e.g. 0000:1b:00.0."""
    return "%04x:%02x:%02x.%x" % (domain, bus, device, function)


def numa_node_of_pci_device(bdf: str, sysfs_root: str = "/sys") -> int:
    """NUMA node of a PCI device as the kernel reports it; -1 when unknown (single-socket hosts often say -1)."""
    import os
    try:
        with open(os.path.join(sysfs_root, "bus", "pci", "devices", bdf.lower(), "numa_node")) as f:
            return int(f.read().strip())
    except (OSError, ValueError):
        return -1


def parse_cpulist(text: str) -> List[int]:
    """'0-3,8,10-11' -> [0, 1, 2, 3, 8, 10, 11]."""
    cpus: List[int] = []
    for part in text.strip().split(","):
        part = part.strip()
        if not part:
            continue
        if "-" in part:
            a, b = part.split("-")
            cpus.extend(range(int(a), int(b) + 1))
        else:
            cpus.append(int(part))
    return sorted(set(cpus))


def cpus_of_numa_node(node: int, sysfs_root: str = "/sys") -> List[int]:
    import os
    if node < 0:
        return []
    try:
        with open(os.path.join(sysfs_root, "devices", "system", "node", "node%d" % node, "cpulist")) as f:
            return parse_cpulist(f.read())
    except (OSError, ValueError):
        return []


def bind_to_numa_node_of(bdf: str, sysfs_root: str = "/sys", apply: bool = True) -> Dict[str, object]:
    """Restricts the calling process (and the threads it starts afterwards) to the CPUs of the PCI device's NUMA
    node, intersected with the CPUs it may already use.  Returns {"numa_node", "cpus", "bound"}; leaves the
    affinity alone when the node is unknown or the intersection is empty."""
    import os
    node = numa_node_of_pci_device(bdf, sysfs_root)
    cpus = cpus_of_numa_node(node, sysfs_root)
    allowed = sorted(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else []
    usable = [c for c in cpus if c in allowed]
    bound = False
    if apply and usable and hasattr(os, "sched_setaffinity"):
        os.sched_setaffinity(0, usable)
        bound = True
    return {"numa_node": node, "cpus": usable, "bound": bound}
