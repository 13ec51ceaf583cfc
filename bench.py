#!/usr/bin/env python
"""Benchmark of the AVSG per-decode-step operator on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Workload: configuration C3 (32 requests x 4 layers = 128 tables, context 131072, top-K 2048, 8192-slot
buffers, 2 query tokens per iteration, 656-byte rows, ~11 GB of pinned host KV).  One "step" is one decode
iteration of the whole batch: four operator calls (one per layer, 32 tables each), every call running
match + reserve (Stage One) and the balanced miss-only host->device gather (Stage Two).

Prints ONE JSON line (rank 0).  value = miss bytes the step needed / device time of the step (GB/s, whole job).
roofline = Stage Two alone against the pinned-copy bandwidth measured in the same run (the host link bounds it);
roofline_stage_one = Stage One against the measured HBM copy bandwidth.

--impl reference times the CPU oracle (plain C, one thread per table over the host cores) on the same
workload; it is a deliberately slow checker, reported as a baseline.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "miss-only H2D gather GB/s (% of link peak); match+reserve us per decode step"
# DRAM traffic per unit from the ncu capture summarised under profiles/ (dram__bytes_read + dram__bytes_write
# per launch of the one-layer case, divided by the units of that launch); scaled by the units of a launch here.
NCU_XFER_DRAM_BYTES_PER_ROW = 91.0          # 0.94 MB per launch of 10.3 k rows: the written rows stay in L2
NCU_S1_DRAM_BYTES_PER_TABLE = {"hash": 59400.0,     # 1.90 MB per launch of 32 tables
                               "direct": 174000.0}  # 5.57 MB: the 2-byte index entries arrive as 32-byte sectors
PAPER_CONTEXT = {
    "hardware": "Ascend 910B NPU (paper), not comparable",
    "hash_vs_dual_pointer_speedup": 2.80, "stage_one_us_K2048_S2048": 53.7,
    "max_h2d_gain_over_request_level": 34.44, "hit_rate_8k_buffer_pct": 94.83,
}


def _measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def _workload(rank: int, n_iters: int, args=None, world: int = 1):
    """C3 for this rank.  Weak scaling (default): every rank has its own full set of tables (its own seed).
    Strong scaling: the ONE set of tables of a single-GPU run is split by request over the ranks
    (sharding.tables_of_rank), every rank keeping all layers of its requests."""
    import dataclasses
    import avsg_traces as tr
    from paper_2609_37538_b200.sharding import tables_of_rank
    kw = {}
    if args is not None:
        kw = {"requests": args.requests, "layers": args.layers}
        if getattr(args, "buffer_slots", 0):
            kw["buffer_slots"] = args.buffer_slots
        if getattr(args, "n_tokens", 0):
            kw["n_q"] = args.n_tokens
    if args is None or getattr(args, "scaling", "weak") == "weak" or world == 1:
        return tr.workload("C3", seed=3 + 1000 * rank, n_iters=n_iters, **kw)
    w = tr.workload("C3", seed=3, n_iters=n_iters, **kw)
    n_req = len(w.calls[0])
    mine = tables_of_rank(n_req, world, rank)                 # requests of this rank
    keep = [grp[r] for grp in w.calls for r in mine]          # their tables, layer by layer
    local = {t: i for i, t in enumerate(keep)}
    calls = [[local[grp[r]] for r in mine] for grp in w.calls]
    return dataclasses.replace(w, tables=[w.tables[t] for t in keep], calls=[c for c in calls if c])


def _gen_traces(w, threads):
    import avsg_traces as tr
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(lambda c: tr.generate(c), w.tables))


# ------------------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle on the host cores
# ------------------------------------------------------------------------------------------------------------
def oracle_run(w, traces, kv_np, tables, warmup, steps, threads, row_stride=None):
    """Steps the oracle over `tables` for warmup+steps iterations, one thread per table; times the last `steps`.
    Returns (seconds per step list, miss rows per step list, hits, misses)."""
    from oracle import OracleTable
    orc = {ti: OracleTable(w.buffer_slots, w.row_bytes, w.max_lifetime) for ti in tables}

    def one(ti, t):
        X, N = traces[ti]
        r = orc[ti].step(X[t], int(N[t]), kv_np[ti], row_stride)
        return int(r.n.sum()), int(r.M.sum())

    secs, rows, hits, misses = [], [], 0, 0
    with ThreadPoolExecutor(max_workers=threads) as ex:
        for t in range(warmup + steps):
            t0 = time.perf_counter()
            res = list(ex.map(lambda ti: one(ti, t), tables))
            dt = time.perf_counter() - t0
            if t >= warmup:
                secs.append(dt)
                rows.append(sum(r[0] for r in res))
                misses += sum(r[0] for r in res)
                hits += sum(r[1] for r in res)
    return secs, rows, hits, misses


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import __graft_entry__
    import avsg_traces as tr
    import oracle
    tr.build_library(); oracle.build_library()
    cores = os.cpu_count() or 1
    n_iters = max(64, args.warmup + args.steps)
    w = _workload(0, n_iters, args)
    traces = _gen_traces(w, cores)
    kv_np = []
    for ti, cfg in enumerate(w.tables):
        a = np.empty(cfg.context * w.row_bytes, np.uint8)
        tr.fill_kv(a, w.seed, ti, cfg.context, w.row_bytes)
        kv_np.append(a)
    tables = list(range(w.num_tables))
    secs, rows, hits, misses = oracle_run(w, traces, kv_np, tables, args.warmup, args.steps, cores)
    total_bytes = sum(rows) * w.row_bytes
    value = total_bytes / 1e9 / sum(secs)
    sample = "all %d tables, %d iterations after %d warm-up, one thread per table over %d threads" % (
        w.num_tables, args.steps, args.warmup, cores)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32/u8",
        "data": "synthetic", "config": _config(w),
        "hit_rate": hits / max(1, hits + misses),
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def _config(w):
    return {"workload": "C3: %d tables (%d requests x %d layers), context 131072, top-K %d, %d-slot buffers, "
                        "%d query tokens per iteration, %d-byte rows, Beta(18,2) overlap; one step = %d calls of %d tables"
                        % (w.num_tables, len(w.calls[0]), len(w.calls), w.topk, w.buffer_slots, w.n_q, w.row_bytes,
                           len(w.calls), len(w.calls[0])),
            "tables": w.num_tables, "topk": w.topk, "buffer_slots": w.buffer_slots, "n_tokens": w.n_q,
            "row_bytes": w.row_bytes, "max_lifetime": w.max_lifetime,
            "host_kv_gb": round(w.host_kv_bytes() / 1e9, 2),
            "l2": "flushed between timed steps (256 MiB write); host KV (11 GB) is far larger than L2"}


# ------------------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------------------
def run_cuda(args):
    import torch
    import torch.distributed as dist
    import __graft_entry__
    import avsg_traces as tr

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    # the rank's threads (trace generation, the fill of the pinned host KV: first touch decides where its pages
    # live) run on the CPUs of the GPU's NUMA node; on by default when there are several ranks
    from paper_2609_37538_b200.sharding import bind_to_numa_node_of, pci_address
    props = torch.cuda.get_device_properties(local)
    bdf = pci_address(getattr(props, "pci_domain_id", 0), getattr(props, "pci_bus_id", 0), getattr(props, "pci_device_id", 0))
    numa = bind_to_numa_node_of(bdf, apply=args.numa_bind == "on" or (args.numa_bind == "auto" and world > 1))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.barrier()
    import paper_2609_37538_b200 as avsg
    avsg.load_library()

    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    threads = max(1, cores if numa["bound"] else cores // world)
    W, K = args.warmup, args.steps
    n_iters = max(64, W + K)
    w = _workload(rank, n_iters, args, world)
    traces = _gen_traces(w, threads)
    kv = []
    stride = args.row_stride or w.row_bytes
    for ti, cfg in enumerate(w.tables):
        buf = avsg.pinned_empty(cfg.context * stride, huge_pages=args.host_kv == "huge")
        tr.fill_kv(buf.data_ptr(), w.seed, ti, cfg.context, w.row_bytes, row_stride=stride)
        kv.append(buf)

    direct = args.index == "direct"
    ctx = avsg.Context(num_tables=w.num_tables, buffer_slots=w.buffer_slots, row_bytes=w.row_bytes,
                       max_topk=w.topk, max_tokens=w.n_q, max_lifetime=w.max_lifetime, device=local,
                       index_mode=avsg.INDEX_DIRECT if direct else avsg.INDEX_HASH,
                       max_context=max(c.context for c in w.tables) + w.n_q, stage_one_cluster=args.cluster,
                       transfer_mode=avsg.XFER_SM_OVERLAP if args.stage_two == "overlap" else avsg.XFER_SM_BALANCED)
    ncalls = len(w.calls)
    calls = [ctx.prepare(grp, [kv[t] for t in grp], w.n_q, w.topk,
                         [stride] * len(grp) if args.row_stride else None) for grp in w.calls]
    # inputs resident in HBM: every iteration's ids, per call [n, n_q, K]
    Xh = [[np.stack([traces[ti][0][t] for ti in grp]) for grp in w.calls] for t in range(n_iters)]
    vlen = [[[int(traces[ti][1][t]) for ti in grp] for grp in w.calls] for t in range(n_iters)]
    Xd = [[torch.from_numpy(x).cuda() for x in row] for row in Xh]
    slots_d = [torch.empty_like(Xd[0][c]) for c in range(ncalls)]
    mc_d = [torch.empty((len(w.calls[c]), w.n_q), dtype=torch.int32, device="cuda") for c in range(ncalls)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def device_step(t):
        for c in range(ncalls):
            calls[c].run(Xd[t][c], vlen[t][c], slots_d[c], None, mc_d[c], stream)

    # ---- host-link peak: large pinned copy on this machine, this run ----
    big_h = torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
    big_d = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    big_d.copy_(big_h, non_blocking=True)
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(4):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); big_d.copy_(big_h, non_blocking=True); e1.record()
        torch.cuda.synchronize()
        best = max(best, (1 << 30) / 1e9 / (e0.elapsed_time(e1) / 1e3))
    link_peak = best
    del big_h, big_d

    # ---- warm-up (cold start + W-1 iterations), then the timed steps ----
    # the first warm-up step is the COLD step (empty buffers: every id misses); it is timed on its own
    flush.fill_(0)
    ce0, ce1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ce0.record()
    device_step(0)
    ce1.record()
    torch.cuda.synchronize()
    cold_ms, cold_rows = ce0.elapsed_time(ce1), ctx.stats()["rows_copied"]
    for t in range(1, W):
        device_step(t)
    torch.cuda.synchronize()
    st0 = ctx.stats()
    ts0 = [ctx.table_stats(ti) for ti in range(w.num_tables)]
    ctx.save_state()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()

    sampler = ClockSampler(local)
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    torch.cuda.synchronize()
    for k in range(K):
        flush.fill_(k & 0xFF)
        ev[k][0].record()
        device_step(W + k)
        ev[k][1].record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    step_ms = [a.elapsed_time(b) for a, b in ev]
    st1 = ctx.stats()
    rows_timed = st1["rows_copied"] - st0["rows_copied"]
    hits_timed, miss_timed = st1["hits"] - st0["hits"], st1["misses"] - st0["misses"]
    # request-level (macro) hit rate: one rate per request over its layers' tables, then the mean over requests
    ts1 = [ctx.table_stats(ti) for ti in range(w.num_tables)]
    req_rates = []
    for r in range(len(w.calls[0])):
        tabs = [grp[r] for grp in w.calls]
        h = sum(ts1[ti]["hits"] - ts0[ti]["hits"] for ti in tabs)
        m = sum(ts1[ti]["misses"] - ts0[ti]["misses"] for ti in tabs)
        req_rates.append(h / max(1, h + m))
    total_ms = sum(step_ms)

    # ---- the same steps once more without the L2 flush (extra figure: the tables' state, 38 MB, stays in L2) ----
    ctx.restore_state()
    torch.cuda.synchronize()
    ev3 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for k in range(K):
        ev3[k][0].record()
        device_step(W + k)
        ev3[k][1].record()
    torch.cuda.synchronize()
    warm_ms = sum(a.elapsed_time(b) for a, b in ev3)

    # ---- the same steps with ALL tables in ONE call per step (extra figure: what the fixed cost of a call weighs;
    # ---- Stage One then serves the tables in rounds while the transfer already copies the earlier rounds' misses) ----
    one_ms = None
    if ncalls > 1 and w.num_tables <= 1024:
        all_tables = [t for grp in w.calls for t in grp]
        call_all = ctx.prepare(all_tables, [kv[t] for t in all_tables], w.n_q, w.topk,
                               [stride] * len(all_tables) if args.row_stride else None)
        X_all = [torch.cat(Xd[W + k]) for k in range(K)]
        v_all = [[v for c in vlen[W + k] for v in c] for k in range(K)]
        slots_all = torch.empty_like(X_all[0])
        ctx.restore_state()
        torch.cuda.synchronize()
        rows_before = ctx.stats()["rows_copied"]
        ev4 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for k in range(K):
            flush.fill_(k & 0xFF)
            ev4[k][0].record()
            call_all.run(X_all[k], v_all[k], slots_all, None, None, stream)
            ev4[k][1].record()
        torch.cuda.synchronize()
        one_ms = sum(a.elapsed_time(b) for a, b in ev4)
        assert ctx.stats()["rows_copied"] - rows_before == rows_timed               # the same misses as the timed steps
        del X_all, slots_all

    # ---- end to end: ids from pinned host memory, slot table back to pinned host memory ----
    Xp = [[torch.from_numpy(x).pin_memory() for x in row] for row in Xh[W:W + K]]
    slots_h = [torch.empty(Xd[0][c].shape, dtype=torch.int32, pin_memory=True) for c in range(ncalls)]
    mc_h = [torch.empty((len(w.calls[c]), w.n_q), dtype=torch.int32, pin_memory=True) for c in range(ncalls)]
    ctx.restore_state()
    torch.cuda.synchronize()
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for k in range(K):
        flush.fill_(k & 0xFF)
        ev2[k][0].record()
        for c in range(ncalls):
            calls[c].run(Xp[k][c], vlen[W + k][c], slots_h[c], None, mc_h[c], stream, host=True)
        ev2[k][1].record()
    torch.cuda.synchronize()
    e2e_ms = sum(a.elapsed_time(b) for a, b in ev2)
    ids_bytes = sum(x.numel() * 4 for x in Xp[0])
    mc_bytes = sum(m.numel() * 4 for m in mc_h)

    # ---- per-kernel times (events inside the library around Stage One / Stage Two), L2 flushed per call ----
    ctx.restore_state()
    ctx.set_transfer_mode(avsg.XFER_SM_BALANCED)      # events between the kernels: one kernel at a time
    ctx.set_timing(True)
    torch.cuda.synchronize()
    ctx.stats()
    s1_us, x_us, x_rows, s1_kus, x_kus = [], [], [], [], []
    for k in range(K):
        for c in range(ncalls):
            flush.fill_(c)
            calls[c].run(Xd[W + k][c], vlen[W + k][c], slots_d[c], None, mc_d[c], stream)
            s = ctx.stats()
            s1_us.append(s["last_stage_one_us"]); x_us.append(s["last_transfer_us"]); x_rows.append(s["last_rows"])
            s1_kus.append(s["last_stage_one_kernel_us"]); x_kus.append(s["last_transfer_kernel_us"])
    # ---- replay of one recorded steady-state call, 1000 times (L2-warm), the paper's Stage One protocol ----
    rep = []
    ctx.save_state()
    for _ in range(args.replays):
        ctx.restore_state()
        calls[0].run(Xd[W + K - 1][0], vlen[W + K - 1][0], slots_d[0], None, mc_d[0], stream)
        rep.append(ctx.stats()["last_stage_one_us"])
    ctx.set_timing(False)
    clocks = sampler.stop()       # sampled from the first timed step to the last replay

    # ---- aggregate over ranks: device time = max over ranks, work = sum over ranks ----
    from paper_2609_37538_b200.sharding import aggregate
    tmax, tsum = aggregate({"total_ms": total_ms, "e2e_ms": e2e_ms, "xus": sum(x_us), "warm_ms": warm_ms, "cold_ms": cold_ms},
                           {"rows": rows_timed, "xrows": sum(x_rows), "hits": hits_timed, "misses": miss_timed,
                            "cold_rows": cold_rows,
                            "req_rate_sum": sum(req_rates), "req_n": len(req_rates)})
    total_ms_j, e2e_ms_j, xus_j = tmax["total_ms"], tmax["e2e_ms"], tmax["xus"]
    rows_j, xrows_j, hits_j, miss_j = tsum["rows"], tsum["xrows"], tsum["hits"], tsum["misses"]

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    rb = w.row_bytes
    value = rows_j * rb / 1e9 / (total_ms_j / 1e3)
    e2e_value = rows_j * rb / 1e9 / (e2e_ms_j / 1e3)
    hbm_peak, peak_kind = _measured_peaks()
    n_launch = len(x_us)
    x_bytes_per_launch = sum(x_rows) * rb / n_launch
    x_avg_us = sum(x_us) / n_launch
    x_gbs = x_bytes_per_launch / 1e3 / x_avg_us
    # Stage One algorithmic bytes per call: state read + write, ids in, slots out, miss counts, miss list
    n_tab = len(w.calls[0])
    s1_bytes = n_tab * (2 * w.buffer_slots * 5 + 2 * w.n_q * w.topk * 4 + w.n_q * 4 + 32) + 8 * sum(x_rows) / n_launch
    if direct:      # direct index: one 2-byte entry read per id, one written per miss
        s1_bytes += n_tab * w.n_q * w.topk * 2 + 2 * sum(x_rows) / n_launch
    s1_avg_us = sum(s1_us) / len(s1_us)
    s1_gbs = s1_bytes / 1e3 / s1_avg_us

    xfer_alone = {"achieved": x_gbs, "duration_us": x_avg_us}
    if args.stage_two == "overlap":
        # The timed steps run avsg_transfer_overlap_kernel, resident from the start of its call's Stage One: its
        # launch lasts the whole call, so its duration is the CUDA-event time of the timed steps / calls per step.
        call_us = 1e3 * total_ms_j / (K * ncalls)
        call_bytes = rows_j * rb / (K * ncalls * world)
        call_gbs = call_bytes / 1e3 / call_us
        roofline = {"bound": "host_link", "kernel": "avsg_transfer_overlap_kernel", "achieved": call_gbs,
                    "peak": link_peak, "unit": "GB/s", "frac": call_gbs / link_peak,
                    "traffic": NCU_XFER_DRAM_BYTES_PER_ROW * call_bytes / rb,
                    "peak_kind": "measured in this run (pinned cudaMemcpyAsync H2D, 1 GiB, best of 4 after one warm-up copy)", "peak_repeats": 4,
                    "duration_us": call_us,
                    "note": "algorithmic bytes = row_bytes x missed rows per launch; duration = CUDA events around the "
                            "timed steps / launches, i.e. the whole call, the part of Stage One that is not hidden "
                            "included; the same copy loop timed alone (balanced mode, one kernel at a time) is "
                            "roofline_transfer_alone; DRAM traffic scaled from the ncu capture of the one-layer case"}
    else:
        roofline = {"bound": "host_link", "kernel": "avsg_transfer_kernel", "achieved": x_gbs, "peak": link_peak,
                    "unit": "GB/s", "frac": x_gbs / link_peak,
                    "traffic": NCU_XFER_DRAM_BYTES_PER_ROW * sum(x_rows) / n_launch,
                    "peak_kind": "measured in this run (pinned cudaMemcpyAsync H2D, 1 GiB, best of 4 after one warm-up copy)", "peak_repeats": 4, "duration_us": x_avg_us,
                    "note": "same object as roofline_transfer_alone"}
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": total_ms_j / K, "ms_per_step_without_l2_flush": tmax["warm_ms"] / K, "higher_is_better": True,
        "scaling": args.scaling if world > 1 else "weak", "vs_baseline": None,
        "dtype": "int32/u8", "data": "synthetic", "config": _config(w),
        "variant": {"host_row_stride": stride, "stage_one_index": args.index, "stage_two": args.stage_two,
                    "stage_one_cluster": args.cluster, "host_kv": args.host_kv},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "GB/s",
                "h2d_bytes_per_step": int(ids_bytes + rows_timed * rb / K), "d2h_bytes_per_step": int(ids_bytes + mc_bytes),
                "ms_per_step": e2e_ms_j / K,
                "note": "avsg_step_host: ids uploaded from pinned host memory, slot table and miss counts "
                        "downloaded; h2d bytes = ids + missed KV rows"},
        "gpu_launches": 2 * ncalls * K,
        "numa": {"gpu_pci": bdf, "numa_node": numa["numa_node"], "bound": numa["bound"], "cpus": len(numa["cpus"]),
                 "note": "rank 0; the pinned host KV is allocated and filled by threads bound to these CPUs when bound"},
        "hit_rate": hits_j / max(1.0, hits_j + miss_j),
        "hit_rate_request_macro": tsum["req_rate_sum"] / max(1.0, tsum["req_n"]),
        "miss_rows_per_step": rows_j / K / world,
        "link_peak_gbs": link_peak, "link": "PCIe Gen5 x16 (nominal 63 GB/s per direction); peak = best 1 GiB pinned cudaMemcpyAsync H2D in this run",
        "pct_of_link_peak": 100.0 * x_gbs / link_peak,
        "match_reserve_us": {"per_call_mean": s1_avg_us, "per_call_median": statistics.median(s1_us),
                             "per_call_min": min(s1_us), "per_call_max": max(s1_us),
                             "replay_median": statistics.median(rep) if rep else None, "replays": len(rep),
                             "in_kernel_mean": sum(s1_kus) / len(s1_kus),
                             "tables_per_call": n_tab,
                             "note": "per_call_*: L2 flushed before each call; replay_*: one recorded call re-run from a restored state (L2-warm)"},
        "transfer_us": {"per_call_mean": x_avg_us, "per_call_median": statistics.median(x_us),
                        "in_kernel_mean": sum(x_kus) / len(x_kus),
                        "in_kernel_gbs": x_bytes_per_launch / 1e3 / (sum(x_kus) / len(x_kus)),
                        "rows_per_call_mean": sum(x_rows) / n_launch,
                        "note": "per_call_*: CUDA events around the launch (what the roofline uses); in_kernel_*: first "
                                "block's start to last block's end on the GPU's clock, without the launch gap"},
        "roofline": roofline,
        "one_call_per_step": None if one_ms is None or world > 1 else {
            "tables_per_call": w.num_tables, "ms_per_step": one_ms / K,
            "gbs": rows_timed * rb / 1e6 / one_ms, "frac_of_link_peak": rows_timed * rb / 1e6 / one_ms / link_peak,
            "note": "the timed steps again with all tables in ONE call per step instead of one call per layer: same "
                    "tables, same traces, same misses; the fixed cost of a call is paid once per step"},
        "target": {
            "stated": "miss-only gather at >= 0.80 of the measured pinned H2D bandwidth",
            "cold_step": {"rows": tsum["cold_rows"], "ms": tmax["cold_ms"],
                          "gbs": tsum["cold_rows"] * rb / 1e6 / tmax["cold_ms"],
                          "frac": tsum["cold_rows"] * rb / 1e6 / tmax["cold_ms"] / link_peak / world,
                          "note": "first step, empty buffers, all ids miss; whole step (4 calls), CUDA events"},
            "steady_call_stage_two_events": {"frac": x_gbs / link_peak},
            "steady_call_stage_two_in_kernel": {"frac": x_bytes_per_launch / 1e3 / (sum(x_kus) / len(x_kus)) / link_peak},
            "steady_whole_call": {"frac": value / link_peak / world},
            "met": {"cold_step": tsum["cold_rows"] * rb / 1e6 / tmax["cold_ms"] / link_peak / world >= 0.8,
                    "steady_call_stage_two_events": x_gbs / link_peak >= 0.8,
                    "steady_call_stage_two_in_kernel": x_bytes_per_launch / 1e3 / (sum(x_kus) / len(x_kus)) / link_peak >= 0.8},
            "ceiling_note": "SM-issued reads of packed 656-byte rows reach 85.5 % of the copy peak at most on this link "
                            "(bench.py --link-model); an event pair around one launch costs 6-7 us beyond the kernel's span"},
        "roofline_transfer_alone": {"bound": "host_link", "kernel": "avsg_transfer_kernel", "achieved": x_gbs, "peak": link_peak,
                     "unit": "GB/s", "frac": x_gbs / link_peak,
                     "traffic": NCU_XFER_DRAM_BYTES_PER_ROW * sum(x_rows) / n_launch,
                     "peak_kind": "measured in this run (pinned cudaMemcpyAsync H2D, 1 GiB, best of 4 after one warm-up copy)", "peak_repeats": 4,
                     "note": "algorithmic bytes = row_bytes x missed rows per launch; the rows cross the host link and stay "
                             "in L2 after the write, so DRAM traffic (scaled from the ncu capture of the one-layer case) is small; "
                             "timed in balanced mode (one kernel at a time); with --stage-two overlap the timed steps run "
                             "avsg_transfer_overlap_kernel, the same copy loop started per token while Stage One still runs"},
        "roofline_stage_one": {"bound": "hbm", "kernel": ("avsg_stage_one_cluster_kernel<%s>" if w.buffer_slots > 8192 or args.cluster > 1
                                                          else "avsg_stage_one_kernel<%s>") % args.index, "achieved": s1_gbs, "peak": hbm_peak,
                               "unit": "GB/s", "frac": s1_gbs / hbm_peak, "traffic": NCU_S1_DRAM_BYTES_PER_TABLE[args.index] * n_tab,
                               "peak_kind": peak_kind,
                               "bytes_per_launch": s1_bytes},
        "paper_context": PAPER_CONTEXT,
    }
    if world == 1 and not args.no_cpu_baseline:
        kv_np = [k.numpy() for k in kv]
        cb_steps = min(16, K)
        tables = list(range(w.num_tables))
        secs, rows, _, _ = oracle_run(w, traces, kv_np, tables, W, cb_steps, cores, stride)
        one_tables = tables[:8]
        secs1, rows1, _, _ = oracle_run(w, traces, kv_np, one_tables, W, 4, 1, stride)
        line["cpu_baseline"] = {
            "value": sum(rows) * rb / 1e9 / sum(secs), "unit": "GB/s", "cores": cores, "kind": "oracle",
            "ms_per_step": 1e3 * sum(secs) / len(secs),
            "sample": "all %d tables, %d iterations after %d warm-up, one thread per table over %d threads"
                      % (w.num_tables, cb_steps, W, cores),
            "single_thread": {"value": sum(rows1) * rb / 1e9 / sum(secs1), "unit": "GB/s",
                              "ms_per_table_iteration": 1e3 * sum(secs1) / len(secs1) / len(one_tables),
                              "sample": "%d tables, 4 iterations after %d warm-up, one thread" % (len(one_tables), W)}}
    if world == 1 and not args.no_comparators:
        # the three-way comparison of the evaluation on C5, inside the same run: free C3 first
        ctx.close()
        del calls, ctx, kv, Xd, Xp
        torch.cuda.empty_cache()
        line["comparators_c5"] = comparators_c5(avsg, torch, tr, link_peak, tiny=args.tiny)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()



# ------------------------------------------------------------------------------------------------------------
# --suite: the five configurations, hit rates, per-call times and the Stage Two comparators (extra report;
# the default run prints only the one line above)
# ------------------------------------------------------------------------------------------------------------
def _suite_one(avsg, torch, tr, name, mode, mode_name, link_peak, needed_rows=None, huge_pages=False, **kw):
    w = tr.workload(name, **kw)
    cores = os.cpu_count() or 1
    traces = _gen_traces(w, cores)
    kv = []
    for ti, cfg in enumerate(w.tables):
        buf = avsg.pinned_empty(cfg.context * w.row_bytes, huge_pages=huge_pages)
        tr.fill_kv(buf.data_ptr(), w.seed, ti, cfg.context, w.row_bytes)
        kv.append(buf)
    ctx = avsg.Context(num_tables=w.num_tables, buffer_slots=w.buffer_slots, row_bytes=w.row_bytes,
                       max_topk=w.topk, max_tokens=w.n_q, max_lifetime=w.max_lifetime, transfer_mode=mode,
                       index_mode=avsg.INDEX_DIRECT, max_context=max(c.context for c in w.tables) + w.n_q)
    ctx.set_timing(True)
    calls = [ctx.prepare(grp, [kv[t] for t in grp], w.n_q, w.topk) for grp in w.calls]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    per_iter = []
    ctx.stats()
    for t in range(w.n_iters):
        s1 = xf = 0.0
        rows = 0
        for c, grp in enumerate(w.calls):
            X = torch.from_numpy(np.stack([traces[ti][0][t] for ti in grp])).cuda()
            slots = torch.empty_like(X)
            flush.fill_(c)
            calls[c].run(X, [int(traces[ti][1][t]) for ti in grp], slots, None, None, stream)
            st = ctx.stats()
            s1 += st["last_stage_one_us"]; xf += st["last_transfer_us"]; rows += st["last_rows"]
        per_iter.append((s1, xf, rows))
    st = ctx.stats()
    rb = w.row_bytes
    cold = per_iter[0]
    steady = per_iter[max(1, len(per_iter) // 4):]
    moved = sum(r for _, _, r in steady)
    need = moved if needed_rows is None else sum(needed_rows[max(1, len(per_iter) // 4):])
    xf_us = sum(x for _, x, _ in steady)
    out = {
        "suite": name, "transfer_mode": mode_name, "tables": w.num_tables, "calls_per_iter": len(w.calls),
        "host_kv_gb": round(w.host_kv_bytes() / 1e9, 2),
        "iters": w.n_iters, "hit_rate": st["hits"] / max(1, st["hits"] + st["misses"]),
        "cold_iter": {"rows": cold[2], "transfer_us": cold[1], "gbs": cold[2] * rb / 1e3 / max(cold[1], 1e-9),
                      "match_reserve_us": cold[0]},
        "steady": {"rows_per_iter": moved / len(steady), "transfer_us_per_iter": xf_us / len(steady),
                   "raw_gbs": moved * rb / 1e3 / xf_us, "effective_gbs": need * rb / 1e3 / xf_us,
                   "pct_of_link_peak": 100.0 * moved * rb / 1e3 / xf_us / link_peak,
                   "match_reserve_us_per_call": sum(a for a, _, _ in steady) / len(steady) / len(w.calls)},
        "rows_per_iter_list": [r for _, _, r in per_iter],
    }
    ctx.close()
    if huge_pages:
        out["host_kv_pages"] = {"requested": "2 MiB transparent huge pages",
                                "huge_fraction": sum(b.huge_bytes for b in kv) / max(1, sum(b.mapped_bytes for b in kv))}
        for b in kv:
            b.free()
    return out


def _suite_modes(avsg, torch, tr, name, **kw):
    """Device time of one iteration (all its calls; CUDA events around it, L2 flushed before it) in the steady state,
    with Stage Two after Stage One (balanced) and overlapping it, for both Stage One indexes."""
    w = tr.workload(name, **kw)
    traces = _gen_traces(w, os.cpu_count() or 1)
    kv = []
    for ti, cfg in enumerate(w.tables):
        buf = avsg.pinned_empty(cfg.context * w.row_bytes)
        tr.fill_kv(buf.data_ptr(), w.seed, ti, cfg.context, w.row_bytes)
        kv.append(buf)
    T = w.n_iters
    X = [[torch.from_numpy(np.stack([traces[ti][0][t] for ti in grp])).cuda() for grp in w.calls] for t in range(T)]
    V = [[[int(traces[ti][1][t]) for ti in grp] for grp in w.calls] for t in range(T)]
    slots = [torch.empty_like(x) for x in X[0]]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    out = {"suite": "stage_two_modes", "config": name, "us_per_iteration": {}}
    for index, iname in ((avsg.INDEX_DIRECT, "direct"), (avsg.INDEX_HASH, "hash")):
        for mode, mname in ((avsg.XFER_SM_BALANCED, "balanced"), (avsg.XFER_SM_OVERLAP, "overlap")):
            ctx = avsg.Context(num_tables=w.num_tables, buffer_slots=w.buffer_slots, row_bytes=w.row_bytes,
                               max_topk=w.topk, max_tokens=w.n_q, max_lifetime=w.max_lifetime, transfer_mode=mode,
                               index_mode=index, max_context=max(c.context for c in w.tables) + w.n_q)
            calls = [ctx.prepare(grp, [kv[t] for t in grp], w.n_q, w.topk, None) for grp in w.calls]
            us = []
            for t in range(T):
                flush.fill_(t & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for c, call in enumerate(calls):
                    call.run(X[t][c], V[t][c], slots[c], None, None, stream)
                e1.record()
                torch.cuda.synchronize()
                if t >= T // 4:
                    us.append(e0.elapsed_time(e1) * 1e3)
            assert ctx.sync_status() == 0
            out["us_per_iteration"]["%s/%s" % (iname, mname)] = sum(us) / len(us)
            del ctx, calls
    return out


# shrunk shapes for --tiny (K <= 256, at most 4 tables, 6 iterations): what the GPU tests run so that this code
# cannot rot; the numbers they give are not measurements of anything
TINY = {
    "C1": dict(topk=64, buffer_slots=256, n_iters=6, context=2048),
    "C2": dict(topk=256, buffer_slots=1024, n_iters=6, context=8192, recent_window=512),
    "C3": dict(topk=256, buffer_slots=1024, n_iters=6, context=8192, requests=2, layers=2, recent_window=512),
    "C4": dict(topk=256, buffer_slots=1024, n_iters=6, context=16384, requests=4, hot_size=64, hot_range=1024),
    "C5": dict(topk=256, buffer_slots=1024, n_iters=6, requests=4, ctx_lo=512, ctx_hi=8192),
}


def _link_peak(torch, nbytes=1 << 30, repeats=4):
    """Best of `repeats` pinned host -> device copies of nbytes (after one warm-up copy), GB/s."""
    big_h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    big_d = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    best = 0.0
    for i in range(repeats + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); big_d.copy_(big_h, non_blocking=True); e1.record()
        torch.cuda.synchronize()
        if i:
            best = max(best, nbytes / 1e9 / (e0.elapsed_time(e1) / 1e3))
    return best


def comparators_c5(avsg, torch, tr, link_peak, tiny=False):
    """Configuration C5 (load-imbalance stress) under the operator's balanced Stage Two and the two comparators the
    evaluation names: request-level assignment (App. D, S1: one block per request) and transfer-all-K (Sec. 4.1,
    no reuse).  Same traces for all three; steady iterations after the cold one; effective GB/s = bytes of the
    rows the operator NEEDS (the balanced run's misses) over the Stage Two time of the mode."""
    kw = dict(TINY["C5"]) if tiny else dict(n_iters=9)
    out = {"workload": "C5: %s" % ("tiny" if tiny else "64 requests, contexts log-uniform in [4096, 524288], cold + 8 steps")}
    need = None
    for mode, mn in ((avsg.XFER_SM_BALANCED, "balanced"), (avsg.XFER_REQUEST_LEVEL, "request_level"),
                     (avsg.XFER_ALL_K, "transfer_all_k")):
        r = _suite_one(avsg, torch, tr, "C5", mode, mn, link_peak, needed_rows=need, **kw)
        if need is None:
            need = r["rows_per_iter_list"]
            out["host_kv_gb"] = r["host_kv_gb"]
            out["hit_rate"] = r["hit_rate"]
            out["rows_needed_per_iter"] = r["steady"]["rows_per_iter"]
        out[mn] = {"stage_two_us_per_iter": r["steady"]["transfer_us_per_iter"],
                   "effective_gbs": r["steady"]["effective_gbs"], "raw_gbs": r["steady"]["raw_gbs"],
                   "pct_of_link_peak": 100.0 * r["steady"]["effective_gbs"] / link_peak}
    out["balanced_over_request_level"] = out["balanced"]["effective_gbs"] / out["request_level"]["effective_gbs"]
    out["balanced_over_transfer_all_k"] = out["balanced"]["effective_gbs"] / out["transfer_all_k"]["effective_gbs"]
    return out


def run_suite(args):
    import torch
    import __graft_entry__
    import avsg_traces as tr
    __graft_entry__.build()
    import paper_2609_37538_b200 as avsg
    torch.cuda.set_device(0)
    tiny = args.tiny
    best = _link_peak(torch, (64 << 20) if tiny else (1 << 30))
    print(json.dumps({"suite": "link", "link_peak_gbs": best}), flush=True)
    M = avsg
    for name in ("C1", "C2", "C3", "C4", "C5"):
        kw = dict(TINY[name]) if tiny else {}
        r = _suite_one(avsg, torch, tr, name, M.XFER_SM_BALANCED, "sm_balanced", best, **kw)
        need = r.pop("rows_per_iter_list")
        print(json.dumps(r), flush=True)
        if name == "C5":      # the load-imbalance stress: same traces under the comparators
            for mode, mn in ((M.XFER_REQUEST_LEVEL, "request_level"), (M.XFER_ALL_K, "transfer_all_k")):
                r2 = _suite_one(avsg, torch, tr, name, mode, mn, best, needed_rows=need, **kw)
                r2.pop("rows_per_iter_list")
                print(json.dumps(r2), flush=True)
        if name == "C4":      # the widest spread of rows over host memory: the same run with the host KV in huge pages
            r2 = _suite_one(avsg, torch, tr, name, M.XFER_SM_BALANCED, "sm_balanced, host KV from avsg_host_kv_alloc",
                            best, huge_pages=True, **kw)
            r2.pop("rows_per_iter_list")
            print(json.dumps(r2), flush=True)
        if name == "C3":      # copy-engine comparator on a few iterations (one async copy per run of rows)
            kw2 = dict(kw, n_iters=6)
            r2 = _suite_one(avsg, torch, tr, name, M.XFER_COPY_ENGINE, "copy_engine", best, needed_rows=need[:6], **kw2)
            r2.pop("rows_per_iter_list")
            print(json.dumps(r2), flush=True)
    for name, kw in (("C1", {}), ("C2", {}), ("C3", {"n_iters": 32}), ("C4", {"n_iters": 32}), ("C5", {})):
        print(json.dumps(_suite_modes(avsg, torch, tr, name, **(dict(TINY[name]) if tiny else kw))), flush=True)


# ------------------------------------------------------------------------------------------------------------
# --link-model: what the host link gives SM-issued reads of scattered rows, by row size and alignment.  Every case is
# an all-miss step of the operator itself (32 tables x 2048 rows), Stage Two timed from inside the kernel, so the
# figures are the ceiling of the gather for that row geometry on this machine.  Next to each measurement: the 32-byte
# sectors and 128-byte lines a row touches (computed from the addresses) and the prediction of a packet model of
# the link fitted to two of the cases (see LINK_MODEL below).
# ------------------------------------------------------------------------------------------------------------
LINK_MODEL = {
    "text": "time per row = (payload + H x packets) / R.  A read request of an SM covers at most one 128-byte line of host "
            "memory and is answered by its own completion packet(s); a request for part of a line that spans the line's "
            "64-byte midpoint is answered by two.  payload = 32-byte sectors fetched.  H (bytes per packet) and R (raw "
            "rate) are fitted so that aligned full lines (one 128-byte packet each) and one large pinned cudaMemcpyAsync "
            "(256-byte packets) are both reproduced.",
}


def _row_wire_bytes(offset, row_bytes, header):
    """Payload sectors, lines and modelled bytes on the wire for a row at byte `offset` of a 128-byte-aligned buffer."""
    a, b = offset, offset + row_bytes
    sectors = lines = packets = 0
    line = a // 128
    while line * 128 < b:
        lo, hi = max(a, line * 128), min(b, line * 128 + 128)
        s0, s1 = (lo % 128) // 32, ((hi - 1) % 128) // 32           # first and last sector of the line that is read
        sectors += s1 - s0 + 1
        lines += 1
        packets += 1 if (s0 == 0 and s1 == 3) or (s0 // 2 == s1 // 2) else 2
        line += 1
    return sectors, lines, sectors * 32 + header * packets


def run_link_model(args):
    import torch
    import __graft_entry__
    import avsg_traces as tr
    __graft_entry__.build()
    import paper_2609_37538_b200 as avsg
    torch.cuda.set_device(0)
    tiny = args.tiny
    peak = _link_peak(torch, (64 << 20) if tiny else (1 << 30))
    n_tab, K, S, steps = (3, 256, 1024, 3) if tiny else (32, 2048, 8192, 5)
    geos = [(656, 656), (656, 672), (656, 704), (656, 768), (640, 640), (1152, 1152), (2048, 2048), (512, 512),
            (256, 256), (128, 128)]
    if tiny:
        geos = [(656, 656), (656, 768), (1152, 1152)]
    if args.case:                                            # one geometry only (what an ncu capture runs)
        geos = [tuple(int(v) for v in args.case.split(":"))]
    rows = []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    rng = np.random.default_rng(12)
    for rb, stride in geos:
        ctx_len = (steps + 1) * K * (2 if tiny else 8)
        kv = [avsg.pinned_empty(ctx_len * stride) for _ in range(n_tab)]
        for i, b in enumerate(kv):
            tr.fill_kv(b.data_ptr(), 21, i, ctx_len, rb, row_stride=stride)
        ctx = avsg.Context(num_tables=n_tab, buffer_slots=S, row_bytes=rb, max_topk=K, max_tokens=1, max_lifetime=16,
                           index_mode=avsg.INDEX_DIRECT, max_context=ctx_len)
        ctx.set_timing(True)
        call = ctx.prepare(list(range(n_tab)), kv, 1, K, [stride] * n_tab)
        perm = [rng.permutation(ctx_len).astype(np.int32) for _ in range(n_tab)]
        us_k, us_e, sect, line, wire = [], [], 0, 0, 0
        for t in range(steps):
            ids = np.stack([np.sort(perm[i][t * K:(t + 1) * K]) for i in range(n_tab)])[:, None, :]    # never seen: all miss
            X = torch.from_numpy(np.ascontiguousarray(ids)).cuda()
            slots = torch.empty_like(X)
            flush.fill_(t)
            call.run(X, [ctx_len] * n_tab, slots, None, None, stream)
            st = ctx.stats()
            assert st["last_rows"] == n_tab * K
            if t:
                us_k.append(st["last_transfer_kernel_us"]); us_e.append(st["last_transfer_us"])
                for x in ids.ravel()[:: max(1, ids.size // 4096)]:
                    a, b, c = _row_wire_bytes(int(x) * stride % 128, rb, 24)
                    sect += a; line += b; wire += c
        n_s = len(ids.ravel()[:: max(1, ids.size // 4096)]) * (steps - 1)
        ctx.close()
        del kv
        k_us = sum(us_k) / len(us_k)
        rows.append({"link_model": True, "row_bytes": rb, "row_stride": stride, "rows_per_launch": n_tab * K,
                     "in_kernel_us": k_us, "event_us": sum(us_e) / len(us_e), "ns_per_row": 1e3 * k_us / (n_tab * K),
                     "gbs": n_tab * K * rb / 1e3 / k_us, "pct_of_link_peak": 100.0 * n_tab * K * rb / 1e3 / k_us / peak,
                     "sectors_per_row": sect / n_s, "lines_per_row": line / n_s, "wire_bytes_per_row_H24": wire / n_s})
    # the same 656-byte rows, the same number of rows per launch, spread over more and more host memory
    if not args.case:
        for n_t, ctx_len in ((3, 4096), (3, 16384)) if tiny else ((16, 16384), (16, 131072), (16, 1 << 20)):
            rb = stride = 656
            kv = [avsg.pinned_empty(ctx_len * stride) for _ in range(n_t)]
            for i, b in enumerate(kv):
                tr.fill_kv(b.data_ptr(), 22, i, ctx_len, rb)
            ctx = avsg.Context(num_tables=n_t, buffer_slots=S, row_bytes=rb, max_topk=K, max_tokens=1, max_lifetime=16,
                               index_mode=avsg.INDEX_DIRECT, max_context=ctx_len)
            ctx.set_timing(True)
            call = ctx.prepare(list(range(n_t)), kv, 1, K)
            perm = [rng.permutation(ctx_len).astype(np.int32) for _ in range(n_t)]
            us_k = []
            for t in range(steps):
                ids = np.stack([np.sort(perm[i][t * K:(t + 1) * K]) for i in range(n_t)])[:, None, :]
                X = torch.from_numpy(np.ascontiguousarray(ids)).cuda()
                slots = torch.empty_like(X)
                flush.fill_(t)
                call.run(X, [ctx_len] * n_t, slots, None, None, stream)
                st = ctx.stats()
                assert st["last_rows"] == n_t * K
                if t:
                    us_k.append(st["last_transfer_kernel_us"])
            ctx.close()
            del kv
            k_us = sum(us_k) / len(us_k)
            print(json.dumps({"link_model": "span", "row_bytes": rb, "tables": n_t, "host_rows_per_table": ctx_len,
                              "host_span_gb": n_t * ctx_len * stride / 1e9, "rows_per_launch": n_t * K, "in_kernel_us": k_us,
                              "ns_per_row": 1e3 * k_us / (n_t * K), "gbs": n_t * K * rb / 1e3 / k_us,
                              "pct_of_link_peak": 100.0 * n_t * K * rb / 1e3 / k_us / peak}), flush=True)
    if not any(r["row_bytes"] == 1152 for r in rows):
        for r in rows:
            del r["wire_bytes_per_row_H24"]
            print(json.dumps(r), flush=True)
        return
    # fit: R from aligned full lines (the 1152-byte rows: 9 packets of 128 + H), H from the memcpy peak (256 + H per 256)
    full = [r for r in rows if r["row_bytes"] == 1152][0]
    t_line = full["ns_per_row"] / 9.0                                  # ns per (128 + H) bytes
    t_256 = 256.0 / peak                                               # ns per (256 + H) bytes of the copy engine
    H = (128.0 * t_256 - 256.0 * t_line) / (t_line - t_256)
    R = (128.0 + H) / t_line
    print(json.dumps({"link_model": "fit", "link_peak_gbs": peak, "header_bytes_H": H, "raw_rate_gbs_R": R,
                      "model": LINK_MODEL["text"]}), flush=True)
    for r in rows:
        wire = r["sectors_per_row"] * 32 + (r["wire_bytes_per_row_H24"] - r["sectors_per_row"] * 32) / 24.0 * H
        r["model_gbs"] = r["row_bytes"] / (wire / R)
        r["model_pct_of_link_peak"] = 100.0 * r["model_gbs"] / peak
        del r["wire_bytes_per_row_H24"]
        print(json.dumps(r), flush=True)


# ------------------------------------------------------------------------------------------------------------
# --breakdown: where the time of ONE call goes, for calls of different sizes (time marks the kernels take on the
# GPU's own clock when timing is on; the event time of the same call around it)
# ------------------------------------------------------------------------------------------------------------
def run_breakdown(args):
    import torch
    import __graft_entry__
    import avsg_traces as tr
    __graft_entry__.build()
    import paper_2609_37538_b200 as avsg
    torch.cuda.set_device(0)
    tiny = args.tiny
    link_peak = _link_peak(torch, (64 << 20) if tiny else (1 << 30))
    print(json.dumps({"breakdown": "link", "link_peak_gbs": link_peak}), flush=True)
    cases = [("C2", dict(TINY["C2"]) if tiny else dict(n_iters=40)),
             ("C3", dict(TINY["C3"], layers=1) if tiny else dict(requests=5, layers=1, n_iters=40)),
             ("C4", dict(TINY["C4"]) if tiny else dict(n_iters=40)),
             ("C3", dict(TINY["C3"], layers=1, requests=3) if tiny else dict(requests=32, layers=1, n_iters=40))]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    for name, kw in cases:
        w = tr.workload(name, **kw)
        traces = _gen_traces(w, os.cpu_count() or 1)
        kv = []
        for ti, cfg in enumerate(w.tables):
            buf = avsg.pinned_empty(cfg.context * w.row_bytes)
            tr.fill_kv(buf.data_ptr(), w.seed, ti, cfg.context, w.row_bytes)
            kv.append(buf)
        grp = w.calls[0]
        X = [torch.from_numpy(np.stack([traces[ti][0][t] for ti in grp])).cuda() for t in range(w.n_iters)]
        V = [[int(traces[ti][1][t]) for ti in grp] for t in range(w.n_iters)]
        slots = torch.empty_like(X[0])
        for mode, mname in ((avsg.XFER_SM_OVERLAP, "overlap"), (avsg.XFER_SM_BALANCED, "balanced")):
            ctx = avsg.Context(num_tables=w.num_tables, buffer_slots=w.buffer_slots, row_bytes=w.row_bytes,
                               max_topk=w.topk, max_tokens=w.n_q, max_lifetime=w.max_lifetime, transfer_mode=mode,
                               index_mode=avsg.INDEX_DIRECT, max_context=max(c.context for c in w.tables) + w.n_q)
            call = ctx.prepare(grp, [kv[t] for t in grp], w.n_q, w.topk)
            untimed, rows_per = [], []
            prev = ctx.stats()
            # pass 1: the call as it runs in production (no events inside the library), CUDA events around it
            for t in range(w.n_iters):
                flush.fill_(t & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); call.run(X[t], V[t], slots, None, None, stream); e1.record()
                torch.cuda.synchronize()
                st = ctx.stats()
                if t >= w.n_iters // 4:
                    untimed.append(e0.elapsed_time(e1) * 1e3)
                    rows_per.append(st["rows_copied"] - prev["rows_copied"])
                prev = st
            ctx.close()
            # pass 2: the same calls with the time marks on
            ctx = avsg.Context(num_tables=w.num_tables, buffer_slots=w.buffer_slots, row_bytes=w.row_bytes,
                               max_topk=w.topk, max_tokens=w.n_q, max_lifetime=w.max_lifetime, transfer_mode=mode,
                               index_mode=avsg.INDEX_DIRECT, max_context=max(c.context for c in w.tables) + w.n_q)
            ctx.set_timing(True)
            call = ctx.prepare(grp, [kv[t] for t in grp], w.n_q, w.topk)
            marks = {k: [] for k in ("last_copy_start_us", "last_first_row_us", "last_first_block_done_us",
                                     "last_call_kernel_us", "last_stage_one_kernel_us")}
            for t in range(w.n_iters):
                flush.fill_(t & 0xFF)
                call.run(X[t], V[t], slots, None, None, stream)
                st = ctx.stats()
                if t >= w.n_iters // 4 and st["last_rows"] > 0:
                    for k in marks:
                        marks[k].append(st[k])
            ctx.close()
            # pass 3: when are the hits usable?  A second stream waits for the word the call writes at the end of
            # its Stage One (avsg_step_args.stage_one_done), not for the call's stream, and records an event
            hits_at, with_outputs = [], []
            try:
                from cuda.bindings import driver as drv
            except ImportError:
                drv = None
            if drv is not None:
                ctx = avsg.Context(num_tables=w.num_tables, buffer_slots=w.buffer_slots, row_bytes=w.row_bytes,
                                   max_topk=w.topk, max_tokens=w.n_q, max_lifetime=w.max_lifetime, transfer_mode=mode,
                                   index_mode=avsg.INDEX_DIRECT, max_context=max(c.context for c in w.tables) + w.n_q)
                call = ctx.prepare(grp, [kv[t] for t in grp], w.n_q, w.topk)
                side = torch.cuda.Stream()
                word = torch.zeros(1, dtype=torch.int64, device="cuda")
                arriving = torch.empty(X[0].shape, dtype=torch.uint8, device="cuda")
                for t in range(w.n_iters):
                    flush.fill_(t & 0xFF)
                    torch.cuda.synchronize()
                    e0, e1, es = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                    err, = drv.cuStreamWaitValue64(side.cuda_stream, word.data_ptr(), t + 1,
                                                   drv.CUstreamWaitValue_flags.CU_STREAM_WAIT_VALUE_EQ)
                    assert err == drv.CUresult.CUDA_SUCCESS
                    es.record(side)
                    e0.record()
                    call.run(X[t], V[t], slots, None, None, stream, stage_one_done=(word, t + 1), arriving=arriving)
                    e1.record()
                    torch.cuda.synchronize()
                    if t >= w.n_iters // 4:
                        hits_at.append(e0.elapsed_time(es) * 1e3)
                        with_outputs.append(e0.elapsed_time(e1) * 1e3)
                ctx.close()
            mean = lambda v: sum(v) / max(1, len(v))
            rows = mean(rows_per)
            ev, copy_start, first_row = mean(untimed), mean(marks["last_copy_start_us"]), mean(marks["last_first_row_us"])
            first_done, call_k = mean(marks["last_first_block_done_us"]), mean(marks["last_call_kernel_us"])
            print(json.dumps({
                "breakdown": name, "tables": len(grp), "stage_two": mname, "rows_per_call": rows,
                "mb_per_call": rows * w.row_bytes / 1e6, "event_us_per_call": ev,
                "gbs": rows * w.row_bytes / 1e3 / ev, "pct_of_link_peak": 100.0 * rows * w.row_bytes / 1e3 / ev / link_peak,
                "split_us": {"launch_and_event_gap": ev - call_k, "stage_one_exposed": copy_start,
                             "first_row": first_row - copy_start, "copy": first_done - first_row,
                             "tail": call_k - first_done},
                "stage_one_kernel_us": mean(marks["last_stage_one_kernel_us"]), "call_kernel_us": call_k,
                "hits_usable_us": mean(hits_at) if hits_at else None,
                "event_us_per_call_with_early_outputs": mean(with_outputs) if with_outputs else None}), flush=True)
        del kv


# ------------------------------------------------------------------------------------------------------------
# --table3: the Stage Two strategies of App. D on the paper's grid (B x reuse, K = 2048, N_mtp = 0, 1152-byte rows)
# ------------------------------------------------------------------------------------------------------------
def run_table3(args):
    import torch
    import __graft_entry__
    import avsg_traces as tr
    __graft_entry__.build()
    import paper_2609_37538_b200 as avsg
    torch.cuda.set_device(0)
    K, S, RB, CTX, B_MAX = (256, 1024, 1152, 8192, 4) if args.tiny else (2048, 8192, 1152, 131072, 32)
    rng = np.random.default_rng(20260937)
    kv = []
    for ti in range(B_MAX):
        buf = avsg.pinned_empty(CTX * RB)
        tr.fill_kv(buf.data_ptr(), 33, ti, CTX, RB)
        kv.append(buf)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    modes = (("S1_request_level", avsg.XFER_REQUEST_LEVEL), ("S2_position_level", avsg.XFER_POSITION_LEVEL),
             ("S3_miss_level", avsg.XFER_SM_BALANCED))
    for B in ((1, 4) if args.tiny else (1, 2, 4, 8, 16, 32)):
        ctx = avsg.Context(num_tables=B, buffer_slots=S, row_bytes=RB, max_topk=K, max_tokens=1, max_lifetime=16)
        ctx.set_timing(True)
        call = ctx.prepare(list(range(B)), kv[:B], 1, K)
        first = np.stack([np.sort(rng.choice(CTX, K, replace=False)) for _ in range(B)]).astype(np.int32)
        Xa = torch.from_numpy(first[:, None, :]).cuda()
        slots = torch.empty_like(Xa)
        call.run(Xa, [CTX] * B, slots, None, None, stream)          # cold step: the first selection becomes resident
        ctx.save_state()
        torch.cuda.synchronize()
        for reuse in ((0.0, 0.5) if args.tiny else (0.0, 0.25, 0.5, 0.75)):
            keep = int(round(reuse * K))
            sel = []
            for b in range(B):
                kept = rng.choice(first[b], keep, replace=False)
                pool = np.setdiff1d(np.arange(CTX, dtype=np.int32), first[b])
                sel.append(np.sort(np.concatenate([kept, rng.choice(pool, K - keep, replace=False)])))
            Xb = torch.from_numpy(np.stack(sel).astype(np.int32)[:, None, :]).cuda()
            row = {"table3": True, "B": B, "reuse_pct": int(reuse * 100), "rows": B * (K - keep),
                   "bytes": B * (K - keep) * RB}
            for name, mode in modes:
                ctx.set_transfer_mode(mode)
                us = []
                for rep in range(args.replays_table3 + 2):
                    ctx.restore_state()
                    flush.fill_(rep)
                    call.run(Xb, [CTX] * B, slots, None, None, stream)
                    st = ctx.stats()
                    if rep >= 2:
                        us.append(st["last_transfer_us"])
                    assert st["last_rows"] == B * (K - keep) or rep == 0
                med = statistics.median(us)
                row[name + "_us"] = med
                row[name + "_gbs"] = row["bytes"] / 1e3 / med
            row["S3_over_S1"] = row["S3_miss_level_gbs"] / row["S1_request_level_gbs"]
            row["S3_over_S2"] = row["S3_miss_level_gbs"] / row["S2_position_level_gbs"]
            print(json.dumps(row), flush=True)
        ctx.close()


# ------------------------------------------------------------------------------------------------------------
# --sweeps: Stage One latency over K and S (the shapes of the paper's Fig. 3), lifetime ablation (App. A),
# capacity study (App. E protocol) and MTP cold-start reuse (App. E), all on synthetic traces, 1 GPU
# ------------------------------------------------------------------------------------------------------------
def _run_tables(avsg, torch, tr, cfgs, S, L, rb=656, replay=0, warm=None, index_mode=0, probe_retries=0):
    """Steps the given per-table trace recipes through one context (one call per iteration).
    Returns (per-iteration (hits, misses), median Stage One us of `replay` replays of the last step)."""
    n, K, n_q, T = len(cfgs), cfgs[0].topk, cfgs[0].n_q, cfgs[0].n_iters
    traces = [tr.generate(c) for c in cfgs]
    ctxlen = max(c.context for c in cfgs)
    kv = avsg.pinned_empty(ctxlen * rb)                     # the bytes do not matter here: all tables share one
    ctx = avsg.Context(num_tables=n, buffer_slots=S, row_bytes=rb, max_topk=K, max_tokens=n_q, max_lifetime=L,
                       index_mode=index_mode, max_context=ctxlen + n_q, probe_retries=probe_retries)
    call = ctx.prepare(list(range(n)), [kv] * n, n_q, K)
    stream = torch.cuda.current_stream()
    per_iter, prev = [], ctx.stats()
    slots = None
    for t in range(T):
        X = torch.from_numpy(np.stack([traces[i][0][t] for i in range(n)])).cuda()
        slots = torch.empty_like(X)
        vlen = [int(traces[i][1][t]) for i in range(n)]
        if replay and t == T - 1:
            ctx.save_state()
        call.run(X, vlen, slots, None, None, stream)
        st = ctx.stats()
        per_iter.append((st["hits"] - prev["hits"], st["misses"] - prev["misses"]))
        prev = st
    med = None
    if replay:
        ctx.set_timing(True)
        us = []
        for _ in range(replay):
            ctx.restore_state()
            call.run(X, vlen, slots, None, None, stream)
            us.append(ctx.stats()["last_stage_one_us"])
        med = statistics.median(us)
    ctx.close()
    return per_iter, med


def run_sweeps(args):
    import torch
    import __graft_entry__
    import avsg_traces as tr
    __graft_entry__.build()
    import paper_2609_37538_b200 as avsg
    torch.cuda.set_device(0)
    tiny = args.tiny
    CTX = 8192 if tiny else 131072
    KB = 256 if tiny else 2048                 # the top-K of the DSA-shaped sweeps
    SB = 1024 if tiny else 8192                # their pool
    NT = 4 if tiny else 16                     # tables
    WIN = 512 if tiny else 4096

    def recipe(table, K, n_q, T, ctx=CTX, seed=77, **kw):
        base = dict(beta=(18, 2), p_recent=0.5, recent_window=WIN)
        base.update(kw)
        return tr.TraceConfig(seed=seed, table=table, topk=K, n_q=n_q, n_iters=T, context=ctx, **base)

    # (a) Stage One latency: S = K = N; K at S = 4096; S at K = 512 (the shapes of the paper's Fig. 3); pools above
    #     8192 slots at K = 2048 (one thread-block cluster per table).  Median of the replays of a steady step.
    if tiny:
        shapes = [("S=K=N", 64, 64), ("K at S=4096", 128, 4096), ("S at K=512", 512, 1024), ("S at K=2048", 2048, 16384)]
    else:
        shapes = [("S=K=N", k, k) for k in (256, 512, 1024, 2048)]
        shapes += [("K at S=4096", k, 4096) for k in (256, 512, 1024, 2048)]
        shapes += [("S at K=512", 512, sz) for sz in (512, 1024, 2048, 4096, 8192)]
        shapes += [("S at K=2048", 2048, sz) for sz in (8192, 16384, 32768)]
    for label, K, S in shapes:
        for B in ((1, 3) if tiny else (1, 32)):
            _, med = _run_tables(avsg, torch, tr, [recipe(i, K, 1, 6 if tiny else 24, ctx=max(CTX, 4 * K)) for i in range(B)],
                                 S, 16, replay=5 if tiny else 300)
            print(json.dumps({"sweep": "stage_one_latency", "series": label, "K": K, "S": S, "tables": B,
                              "match_reserve_us_median": med}), flush=True)
    # (b) lifetime ablation: K = 2048, 8K pool, MTP-0, 16 tables, 200 steps, steady steps only
    T, skip = (6, 2) if tiny else (200, 40)
    for L in ((1, 16) if tiny else (1, 2, 4, 8, 16, 32)):
        per, med = _run_tables(avsg, torch, tr, [recipe(i, KB, 1, T) for i in range(NT)], SB, L, replay=3 if tiny else 100)
        h = sum(a for a, _ in per[skip:]); m = sum(b for _, b in per[skip:])
        print(json.dumps({"sweep": "lifetime", "L": L, "hit_rate": h / (h + m), "match_reserve_us_median": med}),
              flush=True)
    # (c) capacity study: max KV 16K, K = 2048, L = 8, MTP-0, adjacent-step similarity gamma fixed, historical
    #     recall ~ N(mu, 0.01^2); 4K and 8K pools; 5 seeds (one table each); 300 steps, the first 60 not counted
    T, skip = (8, 2) if tiny else (300, 60)
    for gamma in ((0.7,) if tiny else (0.5, 0.7, 0.9)):
        for mu in ((0.7,) if tiny else (0.5, 0.7, 0.9)):
            row = {"sweep": "capacity", "gamma": gamma, "mu_hist": mu}
            for S in ((512, 1024) if tiny else (4096, 8192)):
                cfgs = [tr.TraceConfig(seed=900 + sd, table=sd, topk=KB, n_q=1, n_iters=T, context=8 * KB,
                                       rho_fixed=gamma, p_hist=mu, hist_sigma=0.01) for sd in range(2 if tiny else 5)]
                per, _ = _run_tables(avsg, torch, tr, cfgs, S, 8)
                h = sum(a for a, _ in per[skip:]); m = sum(b for _, b in per[skip:])
                row["hit_rate_%dK" % (S // 1024) if S >= 1024 else "hit_rate_%d" % S] = h / (h + m)
            print(json.dumps(row), flush=True)
    # (e) the paper's Hash-State table as printed (bounded probing, lossy) against the exact indexes
    T, skip = (6, 2) if tiny else (200, 40)
    for n_q in ((2,) if tiny else (1, 2)):
        cfgs = [recipe(i, KB, n_q, T) for i in range(NT)]
        for label, mode, R in (("exact_hash", avsg.INDEX_HASH, 0), ("exact_direct", avsg.INDEX_DIRECT, 0),
                               ("paper_R1", avsg.INDEX_PAPER, 1), ("paper_R3", avsg.INDEX_PAPER, 3),
                               ("paper_R7", avsg.INDEX_PAPER, 7)):
            per, med = _run_tables(avsg, torch, tr, cfgs, SB, 16, replay=3 if tiny else 100, index_mode=mode, probe_retries=R)
            h = sum(a for a, _ in per[skip:]); m = sum(b for _, b in per[skip:])
            print(json.dumps({"sweep": "index_mode", "n_tokens": n_q, "index": label, "hit_rate": h / (h + m),
                              "rows_copied_per_table_iter": m / NT / (T - skip), "match_reserve_us_median": med}), flush=True)
    # (f) what the overlapped Stage Two buys as the MTP degree grows: one 32-table call per iteration, K = 2048,
    #     8K pool, direct index; device time per call (CUDA events, L2 flushed before each), steady iterations
    NB, T, skip = (3, 6, 2) if tiny else (32, 40, 10)
    kvs = [avsg.pinned_empty(CTX * 656) for _ in range(NB)]
    for i, b in enumerate(kvs):
        tr.fill_kv(b.data_ptr(), 77, i, CTX, 656)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    for n_q in ((1, 3) if tiny else (1, 2, 3, 4)):
        cfgs = [recipe(i, KB, n_q, T) for i in range(NB)]
        traces = [tr.generate(c) for c in cfgs]
        X = [torch.from_numpy(np.stack([traces[i][0][t] for i in range(NB)])).cuda() for t in range(T)]
        V = [[int(traces[i][1][t]) for i in range(NB)] for t in range(T)]
        slots = torch.empty_like(X[0])
        row = {"sweep": "overlap_vs_tokens", "n_tokens": n_q}
        for mode, mname in ((avsg.XFER_SM_BALANCED, "balanced"), (avsg.XFER_SM_OVERLAP, "overlap")):
            ctx = avsg.Context(num_tables=NB, buffer_slots=SB, row_bytes=656, max_topk=KB, max_tokens=n_q,
                               max_lifetime=16, transfer_mode=mode, index_mode=avsg.INDEX_DIRECT, max_context=CTX + n_q)
            call = ctx.prepare(list(range(NB)), kvs, n_q, KB)
            us = []
            for t in range(T):
                flush.fill_(t)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); call.run(X[t], V[t], slots, None, None, stream); e1.record()
                torch.cuda.synchronize()
                if t >= skip:
                    us.append(e0.elapsed_time(e1) * 1e3)
            st = ctx.stats()
            row[mname + "_us"] = sum(us) / len(us)
            row["rows_copied_total"] = st["rows_copied"]
            ctx.close()
        print(json.dumps(row), flush=True)
    del kvs
    # (d) MTP cold start: reuse inside the first iteration from an empty buffer, degrees 0..3, 32 tables
    for deg in ((0, 3) if tiny else range(4)):
        per, _ = _run_tables(avsg, torch, tr, [recipe(i, KB, deg + 1, 1) for i in range(NB)], SB, 16)
        h, m = per[0]
        print(json.dumps({"sweep": "mtp_cold_start", "n_mtp": deg, "reuse": h / (h + m),
                          "rows_copied_per_request": m / NB}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--replays", type=int, default=1000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--requests", type=int, default=32, help="requests per layer (32 = the full configuration)")
    ap.add_argument("--layers", type=int, default=4, help="layers (4 = the full configuration)")
    ap.add_argument("--buffer-slots", type=int, default=0,
                    help="slots per table (0 = the configuration's 8192); above 8192 Stage One runs one thread-block "
                         "cluster per table, e.g. --buffer-slots 16384 --n-tokens 4 for an MTP-3 deployment")
    ap.add_argument("--n-tokens", type=int, default=0, help="query tokens per iteration (0 = the configuration's 2)")
    ap.add_argument("--index", default="direct", choices=["hash", "direct"],
                    help="Stage One index: direct-address table in device memory (default) or shared-memory hash table")
    ap.add_argument("--stage-two", default="overlap", choices=["balanced", "overlap"],
                    help="overlap: Stage Two starts on token g's misses while Stage One places token g+1; balanced: it "
                         "starts when Stage One is complete (the per-kernel figures are always taken in balanced mode, "
                         "where an event can separate the two kernels; the copy loop is the same)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: weak = every rank has its own 128 tables (default); strong = the 128 tables of the "
                         "single-GPU run are split by request over the ranks")
    ap.add_argument("--numa-bind", default="auto", choices=["auto", "on", "off"],
                    help="bind the rank to the CPUs of its GPU's NUMA node before the host KV is allocated "
                         "(auto = when there are several ranks)")
    ap.add_argument("--host-kv", default="pinned", choices=["pinned", "huge"],
                    help="host KV from torch's pinned allocator (default) or from avsg_host_kv_alloc with huge pages")
    ap.add_argument("--tiny", action="store_true",
                    help="with --suite / --table3 / --sweeps: shrunk shapes that finish in seconds (what the tests run)")
    ap.add_argument("--no-comparators", action="store_true",
                    help="skip the comparators_c5 object (balanced / request-level / transfer-all-K on C5)")
    ap.add_argument("--cluster", type=int, default=0, choices=[0, 1, 2, 4, 8],
                    help="thread blocks per table in Stage One (0 = the library's choice)")
    ap.add_argument("--row-stride", type=int, default=0,
                    help="bytes between host KV rows (0 = packed, 656); e.g. 768 pads rows to 128-byte lines")
    ap.add_argument("--table3", action="store_true",
                    help="extra report: Stage Two strategies S1/S2/S3 on the paper's B x reuse grid (1 GPU)")
    ap.add_argument("--replays-table3", type=int, default=9)
    ap.add_argument("--sweeps", action="store_true",
                    help="extra report: Stage One K/S latency sweep, lifetime ablation, capacity study, MTP cold start")
    ap.add_argument("--link-model", action="store_true",
                    help="extra report: Stage Two's rate on all-miss steps by row size and alignment, against a packet "
                         "model of the host link (1 GPU)")
    ap.add_argument("--case", default="", help="with --link-model: only this ROW_BYTES:STRIDE geometry")
    ap.add_argument("--breakdown", action="store_true",
                    help="extra report: where the time of one call goes (Stage One exposed, first row, copy, tail, "
                         "launch gap) for calls of 0.2 .. 6 MB (1 GPU)")
    ap.add_argument("--suite", action="store_true",
                    help="extra report: C1..C5 hit rates, per-call times and the Stage Two comparators (1 GPU)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.link_model:
        run_link_model(args)
    elif args.breakdown:
        run_breakdown(args)
    elif args.sweeps:
        run_sweeps(args)
    elif args.table3:
        run_table3(args)
    elif args.suite:
        run_suite(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
