"""Multi-GPU host logic on CPU: two gloo ranks shard the tables, step their shares with the oracle standing in
for the device (the kernels need a GPU), and reduce counters and timings the way bench.py does."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37538_b200.sharding import aggregate, tables_of_rank, whole_job_gbs


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
