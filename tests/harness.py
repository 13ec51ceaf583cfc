"""Runs a workload through the CUDA path and the oracle side by side and compares them bit for bit."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Sequence

import numpy as np

import avsg_traces as tr
from oracle import OracleTable


class HostKV:
    """Pinned host KV of a set of tables, filled by the seeded generator."""

    def __init__(self, w: tr.Workload, tables: Sequence[int], row_stride: Optional[int] = None,
                 huge_pages: bool = False):
        import paper_2609_37538_b200 as avsg
        self.stride = w.row_bytes if row_stride is None else row_stride
        self.t, self.np = {}, {}
        for ti in tables:
            cfg = w.tables[ti]
            buf = avsg.pinned_empty(cfg.context * self.stride, huge_pages=huge_pages)
            if self.stride != w.row_bytes:
                buf.numpy()[:] = 0xEE
            tr.fill_kv(buf.data_ptr(), w.seed, ti, cfg.context, w.row_bytes, row_stride=self.stride)
            self.t[ti] = buf
            self.np[ti] = buf.numpy()


def run_parity(w: tr.Workload, *, tables: Optional[Sequence[int]] = None, mode: int = 0, host_io: bool = False,
               row_stride: Optional[int] = None, buffer_every: int = 1, oracle_tables: Optional[Sequence[int]] = None,
               n_iters: Optional[int] = None, threads: Optional[int] = None, xfer_geometry=None,
               index_mode: int = 0, permute_seed: Optional[int] = None, cluster: int = 0,
               huge_pages: bool = False, signal: bool = False, arriving: bool = False) -> Dict:
    """Steps every call group of w for every iteration on the GPU; the tables in oracle_tables (default: all)
    are stepped by the oracle too and compared after EVERY step: hit mask, slot table, miss counts, (tok, life);
    the buffer rows every buffer_every iterations and at the end.  With permute_seed the K positions of every token
    of every table are shuffled (seeded) before either side sees them, so that position order and id order differ
    (the k-th miss in POSITION order takes the k-th dead slot).  Returns counters of both sides."""
    import torch
    import paper_2609_37538_b200 as avsg

    ids = list(range(w.num_tables)) if tables is None else list(tables)
    check = set(ids if oracle_tables is None else oracle_tables)
    traces = {}
    with ThreadPoolExecutor(max_workers=threads or os.cpu_count()) as ex:
        for ti, res in zip(ids, ex.map(lambda i: tr.generate(w.tables[i]), ids)):
            traces[ti] = res
    if permute_seed is not None:
        for ti in ids:
            X, N = traces[ti]
            rng = np.random.default_rng([permute_seed, ti])
            order = np.argsort(rng.random(X.shape), axis=-1)
            traces[ti] = (np.ascontiguousarray(np.take_along_axis(X, order, axis=-1)), N)
    kv = HostKV(w, ids, row_stride, huge_pages)
    T = w.n_iters if n_iters is None else min(n_iters, w.n_iters)
    local = {ti: k for k, ti in enumerate(ids)}                  # context table id of a workload table
    ctx = avsg.Context(num_tables=len(ids), buffer_slots=w.buffer_slots, row_bytes=w.row_bytes, max_topk=w.topk,
                       max_tokens=w.n_q, max_lifetime=w.max_lifetime, transfer_mode=mode, device=0,
                       index_mode=index_mode, max_context=max(c.context for c in w.tables) + w.n_q,
                       stage_one_cluster=cluster)
    if xfer_geometry:
        ctx.set_transfer_geometry(*xfer_geometry)
    orc = {ti: OracleTable(w.buffer_slots, w.row_bytes, w.max_lifetime) for ti in ids if ti in check}
    calls = [[ti for ti in grp if ti in local] for grp in w.calls]
    calls = [g for g in calls if g]
    pool = ThreadPoolExecutor(max_workers=threads or os.cpu_count())
    all_k = mode == avsg.XFER_ALL_K

    def oracle_step(ti, t):
        X, N = traces[ti]
        if all_k:
            return orc[ti].step_all_k(X[t], kv.np[ti], kv.stride)
        return orc[ti].step(X[t], int(N[t]), kv.np[ti], kv.stride)

    n_signalled = 0
    signal_word = torch.zeros(1, dtype=torch.int64, device="cuda") if signal else None
    try:
        for t in range(T):
            for grp in calls:
                Xh = np.stack([traces[ti][0][t] for ti in grp])
                vlen = [int(traces[ti][1][t]) for ti in grp]
                tids = [local[ti] for ti in grp]
                kvs = [kv.t[ti] for ti in grp]
                strides = [kv.stride] * len(grp) if row_stride is not None else None
                futs = {ti: pool.submit(oracle_step, ti, t) for ti in grp if ti in check}
                if host_io:
                    out = ctx.step_host(tids, torch.from_numpy(Xh).pin_memory(), kvs, vlen, strides)
                    torch.cuda.synchronize()
                    slots, hit, mc = out.slots.numpy(), out.hit.numpy(), out.miss_count.numpy()
                else:
                    if signal:                       # the call announces the end of its Stage One in a word of ours
                        n_signalled += 1
                        out = ctx.step(tids, torch.from_numpy(Xh).cuda(), kvs, vlen, strides,
                                       stage_one_done=(signal_word, n_signalled), want_arriving=arriving)
                    else:
                        out = ctx.step(tids, torch.from_numpy(Xh).cuda(), kvs, vlen, strides, want_arriving=arriving)
                    torch.cuda.synchronize()
                    if signal:
                        assert int(signal_word.item()) == n_signalled, ("signal", w.name, t)
                    slots, hit, mc = out.slots.cpu().numpy(), out.hit.cpu().numpy(), out.miss_count.cpu().numpy()
                arr = out.arriving.cpu().numpy() if arriving and not host_io else None
                for k, ti in enumerate(grp):
                    if ti not in check:
                        continue
                    r = futs[ti].result()
                    if all_k:
                        assert (slots[k] == r).all(), ("slots", w.name, ti, t)
                        continue
                    assert (hit[k] == r.M).all(), ("hit mask", w.name, ti, t)
                    assert (slots[k] == r.O).all(), ("slot table", w.name, ti, t)
                    assert (mc[k] == r.n).all(), ("miss counts", w.name, ti, t)
                    if arr is not None:
                        assert (arr[k] == r.arriving).all(), ("rows that arrive with this call", w.name, ti, t)
                    tok, life = ctx.export_state(local[ti])
                    c, l = orc[ti].export_state()
                    assert (tok == c).all(), ("cached ids", w.name, ti, t)
                    assert (life == l).all(), ("lifetimes", w.name, ti, t)
            if (t + 1) % buffer_every == 0 or t == T - 1:
                for ti in ids:
                    if ti in check:
                        got = ctx.buffer(local[ti]).cpu().numpy()
                        assert (got == orc[ti].rows()).all(), ("buffer rows", w.name, ti, t)
        assert ctx.sync_status() == 0
        st = ctx.stats()
        oc = {k: sum(o.counters()[k] for o in orc.values()) for k in
              ("steps", "tokens", "hits", "misses", "rows_copied", "extra_decays")}
        if not all_k:
            for ti, o in orc.items():                                   # per-table counters (request-level rates)
                ts, c = ctx.table_stats(local[ti]), o.counters()
                for k in oc:
                    assert ts[k] == c[k], ("table counters", w.name, ti, k, ts[k], c[k])
        if check == set(ids):
            if all_k:
                assert st["rows_copied"] == oc["rows_copied"]
            else:
                for k in oc:
                    assert st[k] == oc[k], (k, st[k], oc[k])
                assert st["bytes_copied"] == oc["rows_copied"] * w.row_bytes
        return {"gpu": st, "oracle": oc, "ctx": ctx, "kv": kv, "traces": traces, "local": local}
    finally:
        pool.shutdown()
