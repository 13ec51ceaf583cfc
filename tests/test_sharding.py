"""Multi-GPU host logic on CPU: two gloo ranks shard the tables, step their shares with the oracle standing in
for the device (the kernels need a GPU), and reduce counters and timings the way bench.py does."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37538_b200.sharding import (aggregate, bind_to_numa_node_of, cpus_of_numa_node,
                                            numa_node_of_pci_device, parse_cpulist, pci_address, tables_of_rank,
                                            whole_job_gbs)


def test_tables_of_rank_partitions_exactly():
    for n, w in [(128, 8), (130, 8), (5, 8), (1, 1), (64, 3)]:
        parts = [tables_of_rank(n, w, r) for r in range(w)]
        flat = [t for p in parts for t in p]
        assert flat == list(range(n))
        assert max(map(len, parts)) - min(map(len, parts)) <= 1
    with pytest.raises(ValueError):
        tables_of_rank(4, 2, 2)


def test_aggregate_without_process_group_is_identity():
    t, w = aggregate({"step_ms": 1.5}, {"rows": 10})
    assert t == {"step_ms": 1.5} and w == {"rows": 10}
    assert whole_job_gbs(2e9, 1000.0) == 2.0


def test_numa_helpers_against_a_fake_sysfs_tree(tmp_path):
    """A two-socket host written out as files: GPU 0000:1b:00.0 on node 0, GPU 0000:9c:00.0 on node 1."""
    allowed = sorted(os.sched_getaffinity(0))
    half = max(1, len(allowed) // 2)
    node_cpus = {0: allowed[:half], 1: allowed[half:] or allowed[:1]}
    for bdf, node in (("0000:1b:00.0", 0), ("0000:9c:00.0", 1), ("0000:aa:00.0", -1)):
        d = tmp_path / "bus" / "pci" / "devices" / bdf
        d.mkdir(parents=True)
        (d / "numa_node").write_text("%d\n" % node)
    for node, cpus in node_cpus.items():
        d = tmp_path / "devices" / "system" / "node" / ("node%d" % node)
        d.mkdir(parents=True)
        (d / "cpulist").write_text(",".join(str(c) for c in cpus) + "\n")
    root = str(tmp_path)
    assert pci_address(0, 0x1b, 0) == "0000:1b:00.0" and pci_address(0, 0x9c, 0) == "0000:9c:00.0"
    assert numa_node_of_pci_device("0000:1B:00.0", root) == 0            # sysfs names are lower case
    assert numa_node_of_pci_device("0000:9c:00.0", root) == 1
    assert numa_node_of_pci_device("0000:aa:00.0", root) == -1 and numa_node_of_pci_device("0000:ff:00.0", root) == -1
    assert parse_cpulist("0-3,8,10-11\n") == [0, 1, 2, 3, 8, 10, 11] and parse_cpulist("") == []
    assert cpus_of_numa_node(1, root) == sorted(node_cpus[1]) and cpus_of_numa_node(-1, root) == []
    before = sorted(os.sched_getaffinity(0))
    try:
        info = bind_to_numa_node_of("0000:9c:00.0", root, apply=False)
        assert info == {"numa_node": 1, "cpus": sorted(node_cpus[1]), "bound": False}
        assert sorted(os.sched_getaffinity(0)) == before                  # apply=False only reports
        info = bind_to_numa_node_of("0000:1b:00.0", root)
        assert info["bound"] and sorted(os.sched_getaffinity(0)) == sorted(node_cpus[0])
        info = bind_to_numa_node_of("0000:aa:00.0", root)                 # unknown node: nothing changes
        assert not info["bound"] and sorted(os.sched_getaffinity(0)) == sorted(node_cpus[0])
    finally:
        os.sched_setaffinity(0, before)


def test_strong_scaling_splits_the_single_gpu_workload_by_request():
    """bench.py --scaling strong: the ranks' tables partition the tables of the single-GPU run (same seed, same
    per-table recipes), every rank keeps all layers of its requests, one call per layer."""
    import importlib.util
    import types
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    args = types.SimpleNamespace(requests=6, layers=3, scaling="strong", buffer_slots=0, n_tokens=0)
    single = bench._workload(0, 8, args, world=1)
    assert single.num_tables == 18 and len(single.calls) == 3
    world = 4
    parts = [bench._workload(r, 8, args, world=world) for r in range(world)]
    seen = []
    for w in parts:
        assert len(w.calls) == 3 and all(len(c) == len(w.calls[0]) for c in w.calls)       # every layer, same requests
        assert sorted(t for c in w.calls for t in c) == list(range(w.num_tables))          # local ids, each table once
        seen += [(t.seed, t.table) for t in w.tables]
    assert sorted(seen) == sorted((t.seed, t.table) for t in single.tables)                # a partition of the job
    assert [len(w.calls[0]) for w in parts] == [2, 2, 1, 1]                                # 6 requests over 4 ranks
    weak = [bench._workload(r, 8, types.SimpleNamespace(requests=6, layers=3, scaling="weak", buffer_slots=0,
                                                        n_tokens=0), world=world) for r in range(2)]
    assert weak[0].num_tables == weak[1].num_tables == 18 and weak[0].tables[0].seed != weak[1].tables[0].seed


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import avsg_traces as tr
    from oracle import OracleTable
    w = tr.workload("C3", topk=64, buffer_slots=256, n_iters=6, context=4096, requests=3, layers=2,
                    recent_window=128)
    mine = tables_of_rank(w.num_tables, world, rank)
    rows = 0
    for ti in mine:
        X, N = tr.generate(w.tables[ti])
        o = OracleTable(w.buffer_slots, 16, w.max_lifetime)
        for t in range(X.shape[0]):
            rows += int(o.step(X[t], int(N[t])).n.sum())
    times, work = aggregate({"step_ms": 10.0 * (rank + 1)}, {"rows": rows, "tables": len(mine)})
    dist.barrier()
    out.put((rank, mine, rows, times, work))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_tables_and_reduce():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, rows0, times0, work0), (r1, t1, rows1, times1, work1) = res
    assert t0 + t1 == list(range(6)) and not set(t0) & set(t1)        # every table on exactly one rank
    assert times0 == times1 == {"step_ms": 20.0}                       # max over ranks
    assert work0 == work1 == {"rows": float(rows0 + rows1), "tables": 6.0}
    # the sharded run moves what a single rank would
    import avsg_traces as tr
    from oracle import OracleTable
    w = tr.workload("C3", topk=64, buffer_slots=256, n_iters=6, context=4096, requests=3, layers=2,
                    recent_window=128)
    total = 0
    for ti in range(w.num_tables):
        X, N = tr.generate(w.tables[ti])
        o = OracleTable(w.buffer_slots, 16, w.max_lifetime)
        total += sum(int(o.step(X[t], int(N[t])).n.sum()) for t in range(X.shape[0]))
    assert total == rows0 + rows1
