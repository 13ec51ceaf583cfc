"""Bit-exact parity of the CUDA path (through the C ABI) with the CPU oracle, on a B200."""
import ctypes
import os

import numpy as np
import pytest

import avsg_traces as tr
from oracle import OracleTable

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def avsg():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2609_37538_b200 as m
    m.load_library()
    return m


def _parity(*a, **kw):
    from harness import run_parity
    return run_parity(*a, **kw)


# ---- the five configurations at full size ---------------------------------------------------------------
def test_c1_full(avsg):
    r = _parity(tr.workload("C1"))
    assert r["gpu"]["tokens"] == 16 and r["gpu"]["extra_decays"] == 0


def test_c2_full(avsg):
    r = _parity(tr.workload("C2"), buffer_every=8)
    g = r["gpu"]
    assert g["tokens"] == 256 and g["hits"] + g["misses"] == 256 * 2048


def test_c3_full(avsg):
    # 128 tables (32 requests x 4 layers), 11 GB of pinned host KV; every table checked after every step
    r = _parity(tr.workload("C3"), buffer_every=16)
    g = r["gpu"]
    assert g["tokens"] == 128 * 64 * 2 and g["hits"] + g["misses"] == g["tokens"] * 2048


def test_c4_full(avsg):
    r = _parity(tr.workload("C4"), buffer_every=16)
    assert r["gpu"]["tokens"] == 16 * 64 * 2


def test_c5_full_balanced(avsg):
    r = _parity(tr.workload("C5"), buffer_every=8)
    assert r["gpu"]["tokens"] == 64 * 33


@pytest.mark.parametrize("mode_name", ["XFER_REQUEST_LEVEL", "XFER_ALL_K", "XFER_POSITION_LEVEL"])
def test_c5_comparators(avsg, mode_name):
    r = _parity(tr.workload("C5", n_iters=6), mode=getattr(avsg, mode_name), buffer_every=2)
    assert r["gpu"]["rows_copied"] == r["oracle"]["rows_copied"]


def test_position_level_comparator_with_mtp_padding_and_host_io(avsg):
    w = tr.workload("C3", requests=5, layers=2, n_iters=8, context=32768)
    _parity(w, mode=avsg.XFER_POSITION_LEVEL, buffer_every=2)
    _parity(w, mode=avsg.XFER_POSITION_LEVEL, host_io=True, buffer_every=4)
    w = tr.workload("C5", topk=128, buffer_slots=256, n_iters=6, requests=4, ctx_lo=40, ctx_hi=100)
    _parity(w, mode=avsg.XFER_POSITION_LEVEL)


def test_copy_engine_comparator(avsg):
    _parity(tr.workload("C3", requests=4, layers=2, n_iters=6, context=32768), mode=avsg.XFER_COPY_ENGINE)


# ---- shapes that span several tiles, ragged tails and the degenerate cases ---------------------------------
SHAPES = [
    # name, overrides
    ("C2", dict(topk=37, buffer_slots=128, n_iters=40, context=4096, recent_window=128)),      # odd K
    ("C2", dict(topk=16, buffer_slots=32, n_iters=60, context=512, recent_window=64)),         # smallest S = N_q K
    ("C2", dict(topk=1000, buffer_slots=2048, n_iters=30, context=65536, recent_window=2048)),  # K not a power of two
    ("C2", dict(topk=4096, buffer_slots=8192, n_iters=10, context=65536, recent_window=8192)),  # S = N_q K at max S
    ("C2", dict(topk=2048, buffer_slots=4096, n_iters=24, context=65536, max_lifetime=1)),      # L = 1, S = N_q K
    ("C2", dict(topk=512, buffer_slots=4096, n_iters=40, context=65536, max_lifetime=126)),     # largest L
    ("C4", dict(topk=300, buffer_slots=1024, n_iters=40, context=1 << 16, requests=5, hot_size=64, hot_range=1024)),
    ("C5", dict(topk=256, buffer_slots=256, n_iters=20, requests=7, ctx_lo=512, ctx_hi=8192)),   # S = K, one token
    ("C5", dict(topk=8192, buffer_slots=8192, n_iters=5, requests=2, ctx_lo=20000, ctx_hi=60000)),  # K = S = max
]


@pytest.mark.parametrize("name,kw", SHAPES)
def test_shapes(avsg, name, kw):
    _parity(tr.workload(name, **kw))


def test_more_tables_than_one_launch_takes(avsg):
    w = tr.workload("C5", topk=64, buffer_slots=128, n_iters=6, requests=300, ctx_lo=256, ctx_hi=2048)
    _parity(w, buffer_every=3)


def test_padding_when_context_is_shorter_than_k(avsg):
    w = tr.workload("C5", topk=128, buffer_slots=256, n_iters=6, requests=4, ctx_lo=40, ctx_hi=100)
    r = _parity(w)
    assert r["gpu"]["hits"] + r["gpu"]["misses"] < 4 * 6 * 128
    for mode in (avsg.XFER_ALL_K, avsg.XFER_POSITION_LEVEL, avsg.XFER_REQUEST_LEVEL, avsg.XFER_SM_OVERLAP):
        _parity(w, mode=mode)                                # padded positions: slot -1, nothing moved, in every mode


def test_strided_host_rows_and_host_io(avsg):
    w = tr.workload("C4", topk=256, buffer_slots=1024, n_iters=12, context=1 << 15, requests=3, hot_size=64,
                    hot_range=1024)
    _parity(w, row_stride=1024)
    _parity(w, host_io=True)


def test_host_kv_from_the_library_allocator(avsg):
    """App. G: host KV in ranges from avsg_host_kv_alloc (2 MiB-aligned, huge pages requested, registered)."""
    import ctypes
    w = tr.workload("C4", topk=256, buffer_slots=1024, n_iters=10, context=1 << 15, requests=3, hot_size=64,
                    hot_range=1024)
    _parity(w, huge_pages=True)
    _parity(w, huge_pages=True, row_stride=1024, mode=avsg.XFER_SM_OVERLAP)
    kv = avsg.HostKV(5 << 20, huge_pages=True)
    assert kv.ptr % (2 << 20) == 0 and 0 <= kv.huge_bytes <= 6 << 20
    assert not kv.numpy().any()                                  # starts as zeros
    plain = avsg.HostKV(4096, huge_pages=False)
    assert plain.ptr % (2 << 20) == 0
    lib = avsg.load_library()
    ptr = kv.ptr
    kv.free()
    assert lib.avsg_host_kv_free(ptr) == avsg.EINVAL             # freed already
    kv.free()                                                    # the wrapper's second free is a no-op
    plain.free()


def test_other_row_sizes(avsg):
    for rb in (16, 1152, 4096):
        _parity(tr.workload("C2", topk=128, buffer_slots=512, n_iters=10, context=8192, row_bytes=rb))


def test_transfer_geometries(avsg):
    w = tr.workload("C5", topk=512, buffer_slots=1024, n_iters=5, requests=9, ctx_lo=1024, ctx_hi=8192)
    for geo in [(1, 32), (7, 1024), (148, 128), (600, 256)]:
        _parity(w, xfer_geometry=geo)


# ---- ids that are not ascending: position order and id order differ (Alg. 1 Pass 3: the k-th miss in POSITION
# ---- order takes the k-th dead slot; the input need not be sorted) ---------------------------------------------
UNSORTED_SHAPES = [
    ("C2", dict(topk=37, buffer_slots=128, n_iters=40, context=4096, recent_window=128)),
    ("C2", dict(topk=1000, buffer_slots=2048, n_iters=24, context=65536, recent_window=2048)),
    ("C4", dict(topk=300, buffer_slots=1024, n_iters=30, context=1 << 16, requests=5, hot_size=64, hot_range=1024)),
    ("C5", dict(topk=128, buffer_slots=256, n_iters=8, requests=4, ctx_lo=40, ctx_hi=100)),     # padding lands anywhere
]


@pytest.mark.parametrize("name,kw", UNSORTED_SHAPES)
@pytest.mark.parametrize("index", ["INDEX_HASH", "INDEX_DIRECT"])
@pytest.mark.parametrize("mode", ["XFER_SM_BALANCED", "XFER_SM_OVERLAP", "XFER_REQUEST_LEVEL"])
def test_unsorted_ids_shapes(avsg, name, kw, index, mode):
    _parity(tr.workload(name, **kw), mode=getattr(avsg, mode), index_mode=getattr(avsg, index), permute_seed=7)


def test_unsorted_ids_c2_full(avsg):
    r = _parity(tr.workload("C2"), permute_seed=11, buffer_every=8, index_mode=avsg.INDEX_DIRECT,
                mode=avsg.XFER_SM_OVERLAP)
    assert r["gpu"]["tokens"] == 256
    _parity(tr.workload("C2", n_iters=48), permute_seed=12, buffer_every=8)


def test_unsorted_ids_differ_from_sorted(avsg):
    """The permutation matters: the same selections in ascending order give another slot table (so a kernel that
    ordered the misses by id could not pass the tests above)."""
    w = tr.workload("C2", topk=64, buffer_slots=256, n_iters=3, context=4096, recent_window=256)
    X, N = tr.generate(w.tables[0])
    order = np.argsort(np.random.default_rng([7, 0]).random(X.shape), axis=-1)
    Xp = np.take_along_axis(X, order, axis=-1)
    a, b = OracleTable(w.buffer_slots, 16, w.max_lifetime), OracleTable(w.buffer_slots, 16, w.max_lifetime)
    ra, rb = a.step(X[0], int(N[0])), b.step(Xp[0], int(N[0]))
    slot_of_a = dict(zip(X[0].ravel().tolist(), ra.O.ravel().tolist()))
    slot_of_b = dict(zip(Xp[0].ravel().tolist(), rb.O.ravel().tolist()))
    assert slot_of_a != slot_of_b


# ---- Stage One across a thread-block cluster: the small shapes with forced cluster sizes, and tables above 8192
# ---- slots, which only a cluster holds -----------------------------------------------------------------------
@pytest.mark.parametrize("name,kw", SHAPES)
@pytest.mark.parametrize("cluster", [2, 4, 8])
@pytest.mark.parametrize("index", ["INDEX_HASH", "INDEX_DIRECT"])
def test_cluster_shapes(avsg, name, kw, cluster, index):
    w = tr.workload(name, **kw)
    if w.buffer_slots // cluster < 32:
        with pytest.raises(avsg.AvsgError) as e:
            _parity(w, cluster=cluster, index_mode=getattr(avsg, index))
        assert e.value.code == avsg.EUNSUPPORTED
        return
    mode = avsg.XFER_SM_OVERLAP if cluster == 4 else avsg.XFER_SM_BALANCED
    _parity(w, cluster=cluster, index_mode=getattr(avsg, index), mode=mode, permute_seed=3 if cluster == 2 else None)


BIG_TABLES = [
    ("C2", dict(topk=2048, n_q=4, buffer_slots=16384, n_iters=14, context=131072)),           # MTP-3, S = 2 N_q K
    ("C2", dict(topk=4096, n_q=2, buffer_slots=16384, n_iters=14, context=131072)),
    ("C3", dict(topk=2048, n_q=4, buffer_slots=16384, n_iters=8, context=65536, requests=5, layers=2)),
    ("C2", dict(topk=8192, n_q=2, buffer_slots=16384, n_iters=6, context=131072)),            # S = N_q K
    ("C2", dict(topk=4096, n_q=4, buffer_slots=32768, n_iters=8, context=131072)),
    ("C5", dict(topk=32768, buffer_slots=32768, n_iters=4, requests=2, ctx_lo=70000, ctx_hi=120000)),   # K = S = max
    ("C2", dict(topk=2048, n_q=2, buffer_slots=32768, n_iters=40, context=131072, max_lifetime=3)),
]


@pytest.mark.parametrize("name,kw", BIG_TABLES)
@pytest.mark.parametrize("index", ["INDEX_HASH", "INDEX_DIRECT"])
@pytest.mark.parametrize("mode", ["XFER_SM_BALANCED", "XFER_SM_OVERLAP"])
def test_tables_above_8192_slots(avsg, name, kw, index, mode):
    r = _parity(tr.workload(name, **kw), index_mode=getattr(avsg, index), mode=getattr(avsg, mode), buffer_every=4)
    assert r["gpu"]["rows_copied"] == r["oracle"]["rows_copied"] > 0


def test_cluster_full_c2_c3_and_unsorted(avsg):
    _parity(tr.workload("C2"), cluster=4, index_mode=avsg.INDEX_DIRECT, mode=avsg.XFER_SM_OVERLAP, buffer_every=8)
    _parity(tr.workload("C2", n_iters=48), cluster=2, index_mode=avsg.INDEX_HASH, permute_seed=4, buffer_every=8)
    _parity(tr.workload("C3", n_iters=24), cluster=4, index_mode=avsg.INDEX_DIRECT, mode=avsg.XFER_SM_OVERLAP,
            buffer_every=8)
    _parity(tr.workload("C4", n_iters=16), cluster=4, index_mode=avsg.INDEX_HASH, buffer_every=8, host_io=True)


# ---- Stage Two overlapping Stage One (latency hiding, App. G) ---------------------------------------------------
@pytest.mark.parametrize("name,kw,index", [
    ("C1", {}, "INDEX_HASH"), ("C2", {}, "INDEX_HASH"), ("C2", {}, "INDEX_DIRECT"), ("C3", {}, "INDEX_DIRECT"),
    ("C3", dict(requests=16, layers=2, n_iters=32), "INDEX_HASH"), ("C4", {}, "INDEX_DIRECT"), ("C5", {}, "INDEX_HASH"),
])
def test_overlap_mode_full(avsg, name, kw, index):
    r = _parity(tr.workload(name, **kw), mode=avsg.XFER_SM_OVERLAP, index_mode=getattr(avsg, index), buffer_every=8)
    assert r["gpu"]["rows_copied"] == r["oracle"]["rows_copied"] > 0


@pytest.mark.parametrize("name,kw", SHAPES)
def test_overlap_mode_shapes(avsg, name, kw):
    _parity(tr.workload(name, **kw), mode=avsg.XFER_SM_OVERLAP)


def test_overlap_mode_host_io_strides_geometries_and_fallbacks(avsg):
    w = tr.workload("C4", topk=256, buffer_slots=1024, n_iters=12, context=1 << 15, requests=3, hot_size=64,
                    hot_range=1024)
    _parity(w, mode=avsg.XFER_SM_OVERLAP, host_io=True)
    _parity(w, mode=avsg.XFER_SM_OVERLAP, row_stride=1024, index_mode=avsg.INDEX_DIRECT)
    for geo in [(1, 32), (7, 1024), (600, 256)]:
        _parity(w, mode=avsg.XFER_SM_OVERLAP, xfer_geometry=geo)
    # more tables than one Stage One launch takes run as the balanced mode
    many = tr.workload("C5", topk=64, buffer_slots=128, n_iters=6, requests=300, ctx_lo=256, ctx_hi=2048)
    _parity(many, mode=avsg.XFER_SM_OVERLAP, buffer_every=3)


def test_overlap_mode_four_tokens_and_mode_switches(avsg):
    """MTP-3: four tokens per iteration, i.e. four publish / wait rounds per call; the transfer mode is switched
    between calls, so calls with and without the per-token counters alternate on one context."""
    import torch
    S, K, n_q, T, rb, n = 2048, 384, 4, 12, 656, 3
    w = tr.workload("C5", topk=K, buffer_slots=S, n_iters=n_q * T, requests=n, ctx_lo=20000, ctx_hi=20001, row_bytes=rb)
    traces = [tr.generate(c) for c in w.tables]
    kv, kvn = [], []
    for ti, cfg in enumerate(w.tables):
        b = avsg.pinned_empty(cfg.context * rb)
        tr.fill_kv(b.data_ptr(), w.seed, ti, cfg.context, rb)
        kv.append(b); kvn.append(b.numpy())
    ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=avsg.XFER_SM_OVERLAP)
    orc = [OracleTable(S, rb, 16) for _ in range(n)]
    for t in range(T):
        ctx.set_transfer_mode(avsg.XFER_SM_BALANCED if t % 4 == 3 else avsg.XFER_SM_OVERLAP)
        X = np.stack([traces[ti][0][n_q * t:n_q * (t + 1), 0, :] for ti in range(n)])     # [n, n_q, K]
        N = [w.tables[ti].context for ti in range(n)]
        out = ctx.step(list(range(n)), torch.from_numpy(np.ascontiguousarray(X)).cuda(), kv, N)
        torch.cuda.synchronize()
        slots, hit, mc = out.slots.cpu().numpy(), out.hit.cpu().numpy(), out.miss_count.cpu().numpy()
        for ti in range(n):
            r = orc[ti].step(X[ti], N[ti], kvn[ti], rb)
            assert (slots[ti] == r.O).all() and (hit[ti] == r.M).all() and (mc[ti] == r.n).all(), (t, ti)
            assert (ctx.buffer(ti).cpu().numpy() == orc[ti].rows()).all(), (t, ti)
    assert ctx.sync_status() == 0


@pytest.mark.parametrize("n,n_q,K,S", [(74, 2, 64, 256),       # Stage One on half of a B200's SMs: still overlapped
                                        (75, 2, 64, 256),       # one more table: Stage One serves the tables in rounds of 32
                                        (100, 4, 32, 256),      # four rounds (the last of 4 tables) x four tokens
                                        (600, 1, 16, 64),       # 19 rounds, the large argument block
                                        (128, 2, 64, 256),      # as many tables as the small argument block takes
                                        (5, 8, 96, 1024),       # as many tokens as the overlapped kernel takes
                                        (3, 9, 100, 1024),      # one more: runs as the balanced mode
                                        (129, 1, 32, 64),       # more tables than the small argument block takes
                                        (1030, 1, 16, 32)])     # more than the large one takes: balanced mode, two launches
def test_overlap_mode_limits(avsg, n, n_q, K, S):
    import torch
    T, rb, ctxlen = 10, 48, 6000
    cfgs = [tr.TraceConfig(seed=5, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen, ctx_growth=n_q > 1,
                           beta=(9, 1), p_recent=0.5, recent_window=512) for i in range(n)]
    traces = [tr.generate(c) for c in cfgs]
    kv = avsg.pinned_empty(ctxlen * rb)                 # every table reads the same host rows
    tr.fill_kv(kv.data_ptr(), 5, 0, ctxlen, rb)
    ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=avsg.XFER_SM_OVERLAP, index_mode=avsg.INDEX_DIRECT,
                       max_context=ctxlen + n_q)
    orc = [OracleTable(S, rb, 16) for _ in range(n)]
    word = torch.zeros(1, dtype=torch.int64, device="cuda")
    for t in range(T):
        X = np.stack([traces[i][0][t] for i in range(n)])
        N = [int(traces[i][1][t]) for i in range(n)]
        if t % 2:                                        # every other iteration through the host-buffer entry point
            out = ctx.step_host(list(range(n)), torch.from_numpy(X).pin_memory(), [kv] * n, N)
        else:                                            # ... and these announce the end of their Stage One
            out = ctx.step(list(range(n)), torch.from_numpy(X).cuda(), [kv] * n, N, stage_one_done=(word, 1000 + t),
                           want_arriving=t % 4 == 0)
        torch.cuda.synchronize()
        assert int(word.item()) == 1000 + t - (t % 2), t
        slots, mc = out.slots.cpu().numpy(), out.miss_count.cpu().numpy()
        arr = out.arriving.cpu().numpy() if out.arriving is not None else None
        for i in range(n):
            r = orc[i].step(X[i], N[i], kv.numpy(), rb)
            assert (slots[i] == r.O).all() and (mc[i] == r.n).all(), (t, i)
            assert arr is None or (arr[i] == r.arriving).all(), (t, i)
    for i in range(0, n, max(1, n // 7)):
        assert (ctx.buffer(i).cpu().numpy() == orc[i].rows()).all(), i
    assert ctx.sync_status() == 0


def test_stage_one_done_signal(avsg):
    """Latency hiding (App. G / Sec. 6): a call announces, in a device word of the caller, that its slot table, hit
    mask and miss counts are final.  Every kind of Stage One kernel writes it, in both Stage Two modes; a second
    stream that waits for the value reads the final outputs while nothing orders it after Stage Two."""
    import torch
    from cuda.bindings import driver as drv
    w = tr.workload("C3", topk=256, buffer_slots=1024, n_iters=8, context=8192, requests=3, layers=1, recent_window=512)
    for kw in (dict(), dict(mode=avsg.XFER_SM_OVERLAP), dict(index_mode=avsg.INDEX_DIRECT, mode=avsg.XFER_SM_OVERLAP),
               dict(cluster=2), dict(cluster=4, mode=avsg.XFER_SM_OVERLAP),
               dict(mode=avsg.XFER_REQUEST_LEVEL), dict(mode=avsg.XFER_POSITION_LEVEL)):
        _parity(w, signal=True, **kw)
        _parity(w, signal=True, arriving=True, permute_seed=3, **kw)     # ... and after the `arriving` output
        _parity(w, arriving=True, **kw)                                  # that output without the word
    w4 = tr.workload("C2", topk=128, n_q=4, buffer_slots=512, n_iters=10, context=4096, recent_window=256)
    for kw in (dict(), dict(index_mode=avsg.INDEX_DIRECT, mode=avsg.XFER_SM_OVERLAP), dict(cluster=4)):
        r = _parity(w4, signal=True, arriving=True, **kw)                # MTP-3: hits on the call's own reservations

    n, n_q, K, S, rb, ctxlen, T = 6, 2, 512, 2048, 656, 30000, 6
    cfgs = [tr.TraceConfig(seed=41, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen, ctx_growth=True,
                           beta=(6, 2), p_recent=0.5, recent_window=2048) for i in range(n)]
    traces = [tr.generate(c) for c in cfgs]
    kv = []
    for i in range(n):
        b = avsg.pinned_empty(ctxlen * rb)
        tr.fill_kv(b.data_ptr(), 41, i, ctxlen, rb)
        kv.append(b)
    side = torch.cuda.Stream()
    word = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx = avsg.Context(n, S, rb, K, n_q, 16, index_mode=avsg.INDEX_PAPER)       # the paper-literal kernel writes it too
    for t in range(3):
        X = torch.from_numpy(np.stack([traces[i][0][t] for i in range(n)])).cuda()
        ctx.step(list(range(n)), X, kv, [int(traces[i][1][t]) for i in range(n)], stage_one_done=(word, 7 + t))
        torch.cuda.synchronize()
        assert int(word.item()) == 7 + t
    assert ctx.sync_status() == 0
    ctx.close()
    for mode in (avsg.XFER_SM_BALANCED, avsg.XFER_SM_OVERLAP):
        ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=mode, index_mode=avsg.INDEX_DIRECT, max_context=ctxlen + n_q)
        orc = [OracleTable(S, rb, 16) for _ in range(n)]
        call = ctx.prepare(list(range(n)), kv, n_q, K)
        early_slots = torch.empty((n, n_q, K), dtype=torch.int32, pin_memory=True)
        early_hit = torch.empty((n, n_q, K), dtype=torch.uint8, pin_memory=True)
        for t in range(T):
            X = np.stack([traces[i][0][t] for i in range(n)])
            N = [int(traces[i][1][t]) for i in range(n)]
            Xd = torch.from_numpy(X).cuda()
            slots = torch.empty_like(Xd)
            hit = torch.empty(Xd.shape, dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()
            value = (mode + 1) * 100 + t
            call.run(Xd, N, slots, hit, None, torch.cuda.current_stream(), stage_one_done=(word, value))
            # the consumer: waits for the word, not for the call's stream
            err, = drv.cuStreamWaitValue64(side.cuda_stream, word.data_ptr(), value,
                                           drv.CUstreamWaitValue_flags.CU_STREAM_WAIT_VALUE_EQ)
            assert err == drv.CUresult.CUDA_SUCCESS
            with torch.cuda.stream(side):
                early_slots.copy_(slots, non_blocking=True)
                early_hit.copy_(hit, non_blocking=True)
            side.synchronize()
            torch.cuda.synchronize()
            for i in range(n):
                r = orc[i].step(X[i], N[i], kv[i].numpy(), rb)
                assert (early_slots[i].numpy() == r.O).all() and (early_hit[i].numpy() == r.M).all(), (mode, t, i)
        assert ctx.sync_status() == 0
        # refusals: the host-buffer entry point, a misaligned word
        Xh = torch.from_numpy(X).pin_memory()
        sh = torch.empty(Xh.shape, dtype=torch.int32, pin_memory=True)
        with pytest.raises(avsg.AvsgError) as e:
            call.run(Xh, N, sh, None, None, None, host=True, stage_one_done=(word, 1))
        assert e.value.code == avsg.EINVAL
        with pytest.raises(avsg.AvsgError) as e:
            call.run(Xd, N, slots, None, None, None, stage_one_done=(word.data_ptr() + 4, 1))
        assert e.value.code == avsg.EINVAL
        ctx.close()
    ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=avsg.XFER_ALL_K)
    with pytest.raises(avsg.AvsgError) as e:
        ctx.step(list(range(n)), Xd, kv, N, stage_one_done=(word, 1))
    assert e.value.code == avsg.EINVAL
    ctx.close()


@pytest.fixture(scope="module")
def early_consumer(tmp_path_factory):
    """tests/cuda/early_consumer.cu built into a shared object: a stand-in for an attention kernel."""
    import ctypes
    import subprocess
    from paper_2609_37538_b200 import build as pkg_build
    so = tmp_path_factory.mktemp("consumer") / "early_consumer.so"
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [f for f in pkg_build.NVCC_FLAGS if f != "--use_fast_math"]
    subprocess.check_call([nvcc] + flags + ["-o", str(so), os.path.join(ROOT, "tests", "cuda", "early_consumer.cu")])
    lib = ctypes.CDLL(str(so))
    vp, u32, u64 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64
    lib.launch_early_consumer.argtypes = [vp, u64, vp, vp, vp, vp, u32, u32, vp, u32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.launch_early_consumer.restype = ctypes.c_int
    return lib


@pytest.mark.parametrize("mode_name", ["XFER_SM_OVERLAP", "XFER_SM_BALANCED"])
def test_a_kernel_on_the_same_stream_starts_on_the_hits(avsg, early_consumer, mode_name):
    """Latency hiding (Sec. 6): a consumer kernel launched right behind avsg_step on the same stream, with
    programmatic stream serialization, runs while Stage Two still copies.  It waits for the call's stage_one_done
    word, then holds the final slot table, hit mask and `arriving` mask and reads the row of the first position that is
    NOT arriving (a hit alone does not say so: a later token may hit a slot reserved earlier in the same call, whose
    row is still travelling, Sec. 3.6); only then does it wait for the stream's earlier work (griddepcontrol.wait)
    and read the row of the first arriving position.  All four are compared with the oracle
    or the host KV."""
    import torch
    n, n_q, K, S, rb, ctxlen, T = 16, 2, 2048, 8192, 656, 60000, 6
    cfgs = [tr.TraceConfig(seed=51, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen, ctx_growth=True,
                           beta=(18, 2), p_recent=0.5, recent_window=4096) for i in range(n)]
    traces = [tr.generate(c) for c in cfgs]
    kv = []
    for i in range(n):
        b = avsg.pinned_empty(ctxlen * rb)
        tr.fill_kv(b.data_ptr(), 51, i, ctxlen, rb)
        kv.append(b)
    ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=getattr(avsg, mode_name), index_mode=avsg.INDEX_DIRECT,
                       max_context=ctxlen + n_q)
    orc = [OracleTable(S, rb, 16) for _ in range(n)]
    call = ctx.prepare(list(range(n)), kv, n_q, K)
    dev = dict(device="cuda")
    word = torch.zeros(1, dtype=torch.int64, **dev)
    slots = torch.empty((n, n_q, K), dtype=torch.int32, **dev)
    hit = torch.empty((n, n_q, K), dtype=torch.uint8, **dev)
    slots_early, hit_early = torch.empty_like(slots), torch.empty_like(hit)
    arriving = torch.empty_like(hit)
    hit_row, miss_row = torch.zeros(rb, dtype=torch.uint8, **dev), torch.zeros(rb, dtype=torch.uint8, **dev)
    picked = torch.empty(2, dtype=torch.int32, **dev)
    marks = torch.zeros(4, dtype=torch.int64, **dev)
    status = torch.zeros(1, dtype=torch.int32, **dev)
    stream = torch.cuda.current_stream()
    buf0 = ctx.buffer(0)
    lead = []
    for t in range(T):
        X = np.stack([traces[i][0][t] for i in range(n)])
        N = [int(traces[i][1][t]) for i in range(n)]
        Xd = torch.from_numpy(X).cuda()
        slots_early.fill_(-7); hit_early.fill_(9)
        torch.cuda.synchronize()
        call.run(Xd, N, slots, hit, None, stream, stage_one_done=(word, t + 1), arriving=arriving)
        rc = early_consumer.launch_early_consumer(word.data_ptr(), t + 1, Xd.data_ptr(), slots.data_ptr(), hit.data_ptr(),
                                                  arriving.data_ptr(),
                                                  n * n_q * K, n_q * K, buf0.data_ptr(), rb, slots_early.data_ptr(),
                                                  hit_early.data_ptr(), hit_row.data_ptr(), miss_row.data_ptr(),
                                                  picked.data_ptr(), marks.data_ptr(), status.data_ptr(),
                                                  stream.cuda_stream or None)
        assert rc == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0                              # the consumer's wait did not run out
        for i in range(n):
            r = orc[i].step(X[i], N[i], kv[i].numpy(), rb)
            assert (slots_early[i].cpu().numpy() == r.O).all() and (hit_early[i].cpu().numpy() == r.M).all(), (t, i)
        hit_id, miss_id = (int(v) for v in picked.cpu())
        host0 = kv[0].numpy().reshape(ctxlen, rb)
        if t > 0:
            assert hit_id >= 0
        if hit_id >= 0:
            assert (hit_row.cpu().numpy() == host0[hit_id]).all(), t         # read BEFORE Stage Two was waited for
        assert miss_id >= 0 and (miss_row.cpu().numpy() == host0[miss_id]).all(), t
        t0, t1, t2, t3 = (int(v) for v in marks.cpu())
        assert t0 <= t1 <= t2 <= t3
        lead.append((t3 - t2) / 1e3)       # how long it still had to wait for Stage Two after finishing with the hits:
                                           # tens of microseconds here; a timing, so reported by pytest -s, not asserted
    print("waited for Stage Two after the hits were done, us:", ["%.1f" % v for v in lead])
    assert ctx.sync_status() == 0
    ctx.close()


_FIRST_CALL_SCRIPT = r"""
import sys, time
import numpy as np, torch
from cuda.bindings import driver as drv
import avsg_traces as tr
import paper_2609_37538_b200 as avsg
mode = getattr(avsg, sys.argv[1])
n, n_q, K, S, rb, ctxlen = 3, 2, 64, 256, 48, 3000
kv = avsg.pinned_empty(ctxlen * rb)
tr.fill_kv(kv.data_ptr(), 1, 0, ctxlen, rb)
X = torch.from_numpy(np.stack([tr.generate(tr.TraceConfig(seed=1, table=i, topk=K, n_q=n_q, n_iters=1, context=ctxlen,
                               ctx_growth=True, beta=(9, 1), p_recent=0.5, recent_window=256))[0][0] for i in range(n)])).cuda()
ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=mode, index_mode=avsg.INDEX_DIRECT, max_context=ctxlen + n_q)
side = torch.cuda.Stream()
word = torch.zeros(1, dtype=torch.int64, device="cuda")
torch.cuda.synchronize()
err, = drv.cuStreamWaitValue64(side.cuda_stream, word.data_ptr(), 1, drv.CUstreamWaitValue_flags.CU_STREAM_WAIT_VALUE_EQ)
assert err == drv.CUresult.CUDA_SUCCESS
released = torch.cuda.Event()
released.record(side)
# the process's FIRST call: none of the call's kernels has been launched before
out = ctx.step(list(range(n)), X, [kv] * n, [ctxlen] * n, stage_one_done=(word, 1), want_arriving=sys.argv[2] == "1")
t0 = time.time()
while not released.query() and time.time() - t0 < 20:
    time.sleep(0.001)
assert released.query(), "the waiting stream was not released"
torch.cuda.synchronize()
assert ctx.sync_status() == 0 and int(word.item()) == 1
print("first call ok")
"""


@pytest.mark.parametrize("mode_name,arriving", [("XFER_SM_OVERLAP", 1), ("XFER_SM_BALANCED", 1), ("XFER_SM_OVERLAP", 0)])
def test_first_call_of_a_process_with_a_waiter_already_armed(mode_name, arriving):
    """A stream that already waits for a call's stage_one_done word when the process makes its first call: the
    library has loaded every kernel when the context was created, so no launch has to wait for the device's other
    streams (the runtime loads a kernel at its first use, which may wait for all streams - here forever)."""
    import subprocess
    import sys
    env = dict(os.environ, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", _FIRST_CALL_SCRIPT, mode_name, str(arriving)], cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "first call ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


@pytest.mark.parametrize("cluster", [0, 2])
@pytest.mark.parametrize("mode_name", ["XFER_SM_BALANCED", "XFER_SM_OVERLAP"])
def test_a_captured_call_can_be_replayed(avsg, mode_name, cluster):
    """One avsg_step call captured in a CUDA graph and replayed for the following iterations: the ids and the
    verified lengths (which grow every iteration here) sit in device tensors that are refreshed in place, and the
    kernel arguments hold nothing else that changes from call to call."""
    import torch
    n, n_q, K, S, T, rb, ctxlen = 4, 2, 256, 1024, 12, 656, 20000
    cfgs = [tr.TraceConfig(seed=11, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen, ctx_growth=True,
                           beta=(18, 2), p_recent=0.5, recent_window=2048) for i in range(n)]
    traces = [tr.generate(c) for c in cfgs]
    assert traces[0][1][0] != traces[0][1][1]                 # the verified length does change
    kv = []
    for i in range(n):
        b = avsg.pinned_empty(ctxlen * rb)
        tr.fill_kv(b.data_ptr(), 11, i, ctxlen, rb)
        kv.append(b)
    ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=getattr(avsg, mode_name), index_mode=avsg.INDEX_DIRECT,
                       max_context=ctxlen + n_q, stage_one_cluster=cluster)
    orc = [OracleTable(S, rb, 16) for _ in range(n)]
    call = ctx.prepare(list(range(n)), kv, n_q, K, None)
    X = torch.empty((n, n_q, K), dtype=torch.int32, device="cuda")
    Nd = torch.empty(n, dtype=torch.int32, device="cuda")
    slots = torch.empty_like(X)
    mc = torch.empty((n, n_q), dtype=torch.int32, device="cuda")

    def load(t):
        X.copy_(torch.from_numpy(np.stack([traces[i][0][t] for i in range(n)])))
        Nd.copy_(torch.tensor([int(traces[i][1][t]) for i in range(n)], dtype=torch.int32))
        torch.cuda.synchronize()

    word = torch.zeros(1, dtype=torch.int64, device="cuda")
    arriving = torch.empty((n, n_q, K), dtype=torch.uint8, device="cuda")

    def check(t):
        torch.cuda.synchronize()
        assert int(word.item()) == 5                       # the captured value, written again by every replay
        word.zero_()
        for i in range(n):
            r = orc[i].step(traces[i][0][t], int(traces[i][1][t]), kv[i].numpy(), rb)
            assert (slots[i].cpu().numpy() == r.O).all() and (mc[i].cpu().numpy() == r.n).all(), (t, i)
            assert (arriving[i].cpu().numpy() == r.arriving).all(), (t, i)
            assert (ctx.buffer(i).cpu().numpy() == orc[i].rows()).all(), (t, i)
            tok, life = ctx.export_state(i)
            c, l = orc[i].export_state()
            assert (tok == c).all() and (life == l).all(), (t, i)

    side = torch.cuda.Stream()
    load(0)
    with torch.cuda.stream(side):
        call.run(X, Nd, slots, None, mc, side,             # eager first call: resolves and caches the host pointers
                 stage_one_done=(word, 5), arriving=arriving)
    check(0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):             # three kernels: Stage One, the `arriving` output, Stage Two
        call.run(X, Nd, slots, None, mc, torch.cuda.current_stream(), stage_one_done=(word, 5), arriving=arriving)
    for t in range(1, T):
        load(t)
        graph.replay()
        check(t)
    assert ctx.sync_status() == 0


@pytest.mark.parametrize("mode_name,index_name", [("XFER_SM_BALANCED", "INDEX_HASH"), ("XFER_SM_OVERLAP", "INDEX_DIRECT")])
def test_stream_ordered_reset(avsg, mode_name, index_name):
    """A request leaves the batch: its table is reset by a kernel in stream order, between two steps, with no host
    synchronisation in between; the other tables carry on untouched."""
    import torch
    n, n_q, K, S, T, rb, ctxlen = 3, 2, 128, 512, 12, 48, 8000
    cfgs = [tr.TraceConfig(seed=21, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen, beta=(9, 1), p_recent=0.5,
                           recent_window=1024) for i in range(n)]
    traces = [tr.generate(c) for c in cfgs]
    kv = avsg.pinned_empty(ctxlen * rb)
    tr.fill_kv(kv.data_ptr(), 21, 0, ctxlen, rb)
    ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=getattr(avsg, mode_name),
                       index_mode=getattr(avsg, index_name), max_context=ctxlen + n_q,
                       stage_one_cluster=4 if index_name == "INDEX_HASH" else 0)     # the hash runs also cover a cluster
    orc = [OracleTable(S, rb, 16) for _ in range(n)]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for t in range(T):
            X = np.stack([traces[i][0][t] for i in range(n)])
            if t in (4, 9):                                  # table 1 (then tables 0 and 2) start over
                gone = [1] if t == 4 else [0, 2]
                ctx.reset_async(gone, stream)
                for i in gone:
                    orc[i].reset()
            out = ctx.step(list(range(n)), torch.from_numpy(X).cuda(), [kv] * n, [ctxlen] * n, stream=stream)
            stream.synchronize()
            slots, hit = out.slots.cpu().numpy(), out.hit.cpu().numpy()
            for i in range(n):
                r = orc[i].step(X[i], ctxlen, kv.numpy(), rb)
                assert (slots[i] == r.O).all() and (hit[i] == r.M).all(), (t, i)
                tok, life = ctx.export_state(i)
                c, l = orc[i].export_state()
                assert (tok == c).all() and (life == l).all(), (t, i)
                assert (ctx.buffer(i).cpu().numpy() == orc[i].rows()).all(), (t, i)
                ts, oc = ctx.table_stats(i), orc[i].counters()
                assert ts["hits"] == oc["hits"] and ts["misses"] == oc["misses"] and ts["steps"] == oc["steps"], (t, i)
    assert ctx.sync_status() == 0


def test_overlap_wait_gives_up_and_the_context_stays_usable(avsg):
    """The overlapped transfer kernel launched without its Stage One: every block polls up to its limit, raises
    the status bit, copies nothing and returns; after clearing the status word the context works as before."""
    import time
    import torch
    w = tr.workload("C2", topk=256, buffer_slots=1024, n_iters=8, context=16384, recent_window=1024)
    X, N = tr.generate(w.tables[0])
    kv = avsg.pinned_empty(w.tables[0].context * w.row_bytes)
    tr.fill_kv(kv.data_ptr(), w.seed, 0, w.tables[0].context, w.row_bytes)
    ctx = avsg.Context(1, w.buffer_slots, w.row_bytes, w.topk, w.n_q, 16, transfer_mode=avsg.XFER_SM_OVERLAP)
    orc = OracleTable(w.buffer_slots, w.row_bytes, 16)

    def step(t):
        out = ctx.step([0], torch.from_numpy(X[t][None]).cuda(), [kv], [int(N[t])])
        torch.cuda.synchronize()
        r = orc.step(X[t], int(N[t]), kv.numpy(), w.row_bytes)
        assert (out.slots[0].cpu().numpy() == r.O).all() and (out.hit[0].cpu().numpy() == r.M).all(), t
        assert (ctx.buffer(0).cpu().numpy() == orc.rows()).all(), t

    for t in range(4):
        step(t)
    assert ctx.sync_status() == 0
    before = ctx.buffer(0).cpu().numpy().copy()
    t0 = time.time()
    ctx.probe_wait_limit()
    word = ctx.sync_status()
    assert time.time() - t0 < 10.0
    assert word == avsg.STATUS_WAIT_TIMEOUT, word
    assert (ctx.buffer(0).cpu().numpy() == before).all()
    # the flags of the overlapped mode carry the number of their call, which the kernel that gave up advanced all
    # the same: the next calls run correctly even BEFORE the status word is cleared (it stays set: it is sticky)
    for t in range(4, 6):
        step(t)
    assert ctx.sync_status() == avsg.STATUS_WAIT_TIMEOUT
    ctx.probe_wait_limit()                       # and a second lost Stage One changes nothing about that
    assert ctx.sync_status() == avsg.STATUS_WAIT_TIMEOUT
    ctx.clear_status()
    assert ctx.sync_status() == 0
    for t in range(6, 8):
        step(t)
    assert ctx.sync_status() == 0


@pytest.mark.parametrize("index,cluster", [("INDEX_HASH", 0), ("INDEX_DIRECT", 0), ("INDEX_DIRECT", 2)])
def test_soak_random_subsets_modes_and_token_counts(avsg, index, cluster):
    """300 calls on one context: every call takes a random subset of the tables in a random order, a random number
    of tokens, a random Stage Two mode and either device or host buffers; every table is compared with its own
    oracle after every call it took part in.  Exercises the hand-over flags of the overlapped mode across calls of
    different shapes (a table's flag of an earlier call must never be taken for a current one)."""
    import torch
    rng = np.random.default_rng(77)
    n, S, K, n_q_max, rb, ctxlen, L = 7, 512, 48, 4, 48, 4000, 5
    kv = []
    for i in range(n):
        b = avsg.pinned_empty(ctxlen * rb)
        tr.fill_kv(b.data_ptr(), 31, i, ctxlen, rb)
        kv.append(b)
    ctx = avsg.Context(n, S, rb, K, n_q_max, L, index_mode=getattr(avsg, index), max_context=ctxlen,
                       stage_one_cluster=cluster)
    orc = [OracleTable(S, rb, L) for _ in range(n)]
    prev = [rng.choice(ctxlen, K, replace=False) for _ in range(n)]
    modes = [avsg.XFER_SM_OVERLAP, avsg.XFER_SM_OVERLAP, avsg.XFER_SM_BALANCED, avsg.XFER_REQUEST_LEVEL,
             avsg.XFER_POSITION_LEVEL]
    for call in range(300):
        tabs = [int(t) for t in rng.permutation(n)[: int(rng.integers(1, n + 1))]]
        n_q = int(rng.integers(1, n_q_max + 1))
        ctx.set_transfer_mode(int(rng.choice(modes)))
        X = np.empty((len(tabs), n_q, K), np.int32)
        for a, t in enumerate(tabs):
            for g in range(n_q):                                     # ~85 % overlap with the table's last selection
                keep = rng.choice(prev[t], int(0.85 * K), replace=False)
                pool = np.setdiff1d(np.arange(ctxlen), keep)
                sel = rng.permutation(np.concatenate([keep, rng.choice(pool, K - len(keep), replace=False)]))
                X[a, g] = sel
                prev[t] = sel
        vlen = [ctxlen] * len(tabs)
        if call % 3 == 2:
            out = ctx.step_host(tabs, torch.from_numpy(X).pin_memory(), [kv[t] for t in tabs], vlen)
        else:
            out = ctx.step(tabs, torch.from_numpy(X).cuda(), [kv[t] for t in tabs], vlen)
        torch.cuda.synchronize()
        slots, hit, mc = out.slots.cpu().numpy(), out.hit.cpu().numpy(), out.miss_count.cpu().numpy()
        for a, t in enumerate(tabs):
            r = orc[t].step(X[a], ctxlen, kv[t].numpy(), rb)
            assert (slots[a] == r.O).all() and (hit[a] == r.M).all() and (mc[a] == r.n).all(), (call, t)
            if call % 10 == 9:
                assert (ctx.buffer(t).cpu().numpy() == orc[t].rows()).all(), (call, t)
    for t in range(n):
        tok, life = ctx.export_state(t)
        c, l = orc[t].export_state()
        assert (tok == c).all() and (life == l).all() and (ctx.buffer(t).cpu().numpy() == orc[t].rows()).all(), t
    assert ctx.sync_status() == 0


@pytest.mark.parametrize("n,mode_name", [(6, "XFER_SM_OVERLAP"), (90, "XFER_SM_OVERLAP"), (40, "XFER_SM_BALANCED")])
def test_two_contexts_on_two_streams_at_once(avsg, n, mode_name):
    """Two contexts, each on a stream of its own, issue their calls without waiting for one another: the kernels of
    both share the GPU.  In the overlapped mode the waiting transfer grid of one context must never keep the other's
    Stage One off the SMs (a transfer grid only starts once every block of its own Stage One has started; 90 tables
    take the round-by-round path).  Both are compared with their oracles after every iteration."""
    import torch
    S, K, n_q, rb, ctxlen, T = 512, 64, 2, 656, 5000, 8
    kv = avsg.pinned_empty(ctxlen * rb)
    tr.fill_kv(kv.data_ptr(), 17, 0, ctxlen, rb)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    ctxs, orcs, traces = [], [], []
    for c in range(2):
        ctxs.append(avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=getattr(avsg, mode_name),
                                 index_mode=avsg.INDEX_DIRECT if c == 0 else avsg.INDEX_HASH, max_context=ctxlen + n_q))
        orcs.append([OracleTable(S, rb, 16) for _ in range(n)])
        traces.append([tr.generate(tr.TraceConfig(seed=60 + c, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen,
                                                  ctx_growth=True, beta=(9, 1), p_recent=0.5, recent_window=512))
                       for i in range(n)])
    for t in range(T):
        outs, Xs, Ns = [], [], []
        for c in range(2):
            X = np.stack([traces[c][i][0][t] for i in range(n)])
            N = [int(traces[c][i][1][t]) for i in range(n)]
            Xd = torch.from_numpy(X).cuda()
            Xs.append(X); Ns.append(N)
            outs.append((Xd, None))
        torch.cuda.synchronize()
        for c in range(2):                                # issued back to back, nothing waits in between
            with torch.cuda.stream(streams[c]):
                outs[c] = (outs[c][0], ctxs[c].step(list(range(n)), outs[c][0], [kv] * n, Ns[c], stream=streams[c]))
        torch.cuda.synchronize()
        for c in range(2):
            out = outs[c][1]
            slots, hit, mc = out.slots.cpu().numpy(), out.hit.cpu().numpy(), out.miss_count.cpu().numpy()
            for i in range(n):
                r = orcs[c][i].step(Xs[c][i], Ns[c][i], kv.numpy(), rb)
                assert (slots[i] == r.O).all() and (hit[i] == r.M).all() and (mc[i] == r.n).all(), (t, c, i)
    for c in range(2):
        for i in range(0, n, max(1, n // 5)):
            assert (ctxs[c].buffer(i).cpu().numpy() == orcs[c][i].rows()).all(), (c, i)
        assert ctxs[c].sync_status() == 0
        ctxs[c].close()


def test_two_host_threads_each_with_a_context(avsg):
    """Two host threads, each driving a context and a stream of its own for the whole trace, nothing shared but the
    library and the GPU: both stay bit-exact."""
    import torch
    from concurrent.futures import ThreadPoolExecutor
    n, S, K, n_q, rb, ctxlen, T = 12, 512, 64, 2, 656, 5000, 10
    kv = avsg.pinned_empty(ctxlen * rb)
    tr.fill_kv(kv.data_ptr(), 18, 0, ctxlen, rb)

    def drive(c):
        torch.cuda.set_device(0)
        stream = torch.cuda.Stream()
        ctx = avsg.Context(n, S, rb, K, n_q, 16, transfer_mode=avsg.XFER_SM_OVERLAP,
                           index_mode=avsg.INDEX_DIRECT if c else avsg.INDEX_HASH, max_context=ctxlen + n_q)
        orc = [OracleTable(S, rb, 16) for _ in range(n)]
        traces = [tr.generate(tr.TraceConfig(seed=70 + c, table=i, topk=K, n_q=n_q, n_iters=T, context=ctxlen,
                                             ctx_growth=True, beta=(9, 1), p_recent=0.5, recent_window=512))
                  for i in range(n)]
        with torch.cuda.stream(stream):
            for t in range(T):
                X = np.stack([traces[i][0][t] for i in range(n)])
                N = [int(traces[i][1][t]) for i in range(n)]
                out = ctx.step(list(range(n)), torch.from_numpy(X).cuda(), [kv] * n, N, stream=stream)
                stream.synchronize()
                slots, mc = out.slots.cpu().numpy(), out.miss_count.cpu().numpy()
                for i in range(n):
                    r = orc[i].step(X[i], N[i], kv.numpy(), rb)
                    assert (slots[i] == r.O).all() and (mc[i] == r.n).all(), (c, t, i)
            stream.synchronize()
            for i in range(0, n, 3):
                assert (ctx.buffer(i).cpu().numpy() == orc[i].rows()).all(), (c, i)
        assert ctx.sync_status() == 0
        ctx.close()
        return True

    with ThreadPoolExecutor(max_workers=2) as ex:
        assert all(ex.map(drive, range(2)))


# ---- behaviours ---------------------------------------------------------------------------------------------
def test_regenerated_speculative_row_is_fetched_again(avsg):
    import torch
    rb, S, K, N = 656, 64, 4, 100
    kv = avsg.pinned_empty((N + 4) * rb)
    tr.fill_kv(kv.data_ptr(), 1, 0, N + 4, rb)
    ctx = avsg.Context(1, S, rb, K, 1, 16)
    orc = OracleTable(S, rb, 16)
    X = np.array([[[5, 50, 99, 100]]], dtype=np.int32)
    out = ctx.step([0], torch.from_numpy(X).cuda(), [kv], [N])
    r = orc.step(X[0], N, kv.numpy())
    assert (out.slots.cpu().numpy()[0] == r.O).all()
    tok, life = ctx.export_state(0)
    assert tok[r.O[0, 3]] == -1 and life[r.O[0, 3]] == 16
    tr.fill_kv(kv.data_ptr() + 100 * rb, 1, 0, 1, rb, first_row=100, version=1)    # host regenerates the row
    out = ctx.step([0], torch.from_numpy(X).cuda(), [kv], [N + 1])
    r = orc.step(X[0], N + 1, kv.numpy())
    assert out.hit.cpu().numpy()[0, 0].tolist() == [1, 1, 1, 0] == r.M[0].tolist()
    assert (ctx.buffer(0).cpu().numpy() == orc.rows()).all()
    new_slot = int(out.slots.cpu().numpy()[0, 0, 3])
    assert (ctx.buffer(0).cpu().numpy()[new_slot] == kv.numpy()[100 * rb:101 * rb]).all()


def test_device_resident_kv_and_reset_import_export(avsg):
    import torch
    rb, S, K = 64, 128, 16
    host = np.empty(1000 * rb, np.uint8)
    tr.fill_kv(host, 2, 0, 1000, rb)
    dkv = torch.from_numpy(host).cuda()
    ctx = avsg.Context(2, S, rb, K, 2, 4)
    orc = OracleTable(S, rb, 4)
    rng = np.random.default_rng(0)
    for step in range(10):
        X = np.stack([np.sort(rng.choice(1000, K, replace=False)) for _ in range(2)]).astype(np.int32)
        out = ctx.step([1], torch.from_numpy(X[None]).cuda(), [dkv], [1000])
        r = orc.step(X, 1000, host)
        assert (out.slots.cpu().numpy()[0] == r.O).all()
    assert (ctx.buffer(1).cpu().numpy() == orc.rows()).all()
    assert (ctx.export_state(0)[0] == -1).all()                      # the other table was never touched
    tok, life = ctx.export_state(1)
    ctx.import_state(0, tok, life)                                   # checkpoint / resume into table 0
    X = np.sort(rng.choice(1000, (1, K), replace=False), axis=1).astype(np.int32)
    a = ctx.step([0], torch.from_numpy(X[None]).cuda(), [dkv], [1000])
    b = ctx.step([1], torch.from_numpy(X[None]).cuda(), [dkv], [1000])
    assert (a.slots.cpu() == b.slots.cpu()).all() and (a.hit.cpu() == b.hit.cpu()).all()
    ctx.reset([1])
    tok, life = ctx.export_state(1)
    assert (tok == -1).all() and (life == -1).all() and (ctx.buffer(1).cpu().numpy() == 0).all()
    c = ctx.step([1], torch.from_numpy(X[None]).cuda(), [dkv], [1000])
    assert c.hit.cpu().numpy().sum() == 0 and c.slots.cpu().numpy()[0, 0].tolist() == list(range(K))


def test_save_restore_replays_a_step(avsg):
    import torch
    w = tr.workload("C2", topk=256, buffer_slots=1024, n_iters=8, context=16384, recent_window=512)
    X, N = tr.generate(w.tables[0])
    kv = avsg.pinned_empty(w.tables[0].context * w.row_bytes)
    tr.fill_kv(kv.data_ptr(), w.seed, 0, w.tables[0].context, w.row_bytes)
    ctx = avsg.Context(1, w.buffer_slots, w.row_bytes, w.topk, 2, 16)
    for t in range(6):
        ctx.step([0], torch.from_numpy(X[t][None]).cuda(), [kv], [int(N[t])])
    ctx.save_state()
    first = ctx.step([0], torch.from_numpy(X[6][None]).cuda(), [kv], [int(N[6])])
    state = ctx.export_state(0)
    for _ in range(3):
        ctx.restore_state()
        again = ctx.step([0], torch.from_numpy(X[6][None]).cuda(), [kv], [int(N[6])])
        assert (again.slots.cpu() == first.slots.cpu()).all() and (again.hit.cpu() == first.hit.cpu()).all()
        s2 = ctx.export_state(0)
        assert (s2[0] == state[0]).all() and (s2[1] == state[1]).all()


def test_timing_and_stats(avsg):
    import torch
    w = tr.workload("C2", topk=512, buffer_slots=2048, n_iters=4, context=16384, recent_window=512)
    X, N = tr.generate(w.tables[0])
    kv = avsg.pinned_empty(w.tables[0].context * w.row_bytes)
    tr.fill_kv(kv.data_ptr(), w.seed, 0, w.tables[0].context, w.row_bytes)
    ctx = avsg.Context(1, w.buffer_slots, w.row_bytes, w.topk, 2, 16)
    ctx.set_timing(True)
    for t in range(4):
        ctx.step([0], torch.from_numpy(X[t][None]).cuda(), [kv], [int(N[t])])
    st = ctx.stats()
    assert st["last_stage_one_us"] > 0 and st["last_transfer_us"] > 0
    # the grids timed from inside (first block start to last block end) fit inside the event pairs around them
    assert 0 < st["last_stage_one_kernel_us"] <= st["last_stage_one_us"] + 1.0
    assert 0 < st["last_transfer_kernel_us"] <= st["last_transfer_us"] + 1.0
    assert st["steps"] == 4 and st["tokens"] == 8 and st["hits"] + st["misses"] == 8 * 512
    assert st["bytes_copied"] == st["rows_copied"] * w.row_bytes == st["misses"] * w.row_bytes
    ctx.set_timing(False)
    ctx.step([0], torch.from_numpy(X[3][None]).cuda(), [kv], [int(N[3])])
    st = ctx.stats()
    assert st["last_stage_one_us"] == 0 and st["last_transfer_kernel_us"] == 0 and st["last_stage_one_kernel_us"] == 0


def test_argument_errors(avsg):
    import torch
    ctx = avsg.Context(4, 64, 32, 16, 2, 4)
    kv = avsg.pinned_empty(100 * 32)
    idx = torch.zeros((1, 2, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(avsg.AvsgError) as e:
        ctx.step([4], idx, [kv], [100])                                  # table id out of range
    assert e.value.code == avsg.EINVAL
    with pytest.raises(avsg.AvsgError) as e:
        ctx.step([1, 1], torch.zeros((2, 2, 16), dtype=torch.int32, device="cuda"), [kv, kv], [100, 100])
    assert e.value.code == avsg.EINVAL                                   # duplicate table
    with pytest.raises(avsg.AvsgError) as e:
        ctx.step([0], torch.zeros((1, 2, 40), dtype=torch.int32, device="cuda"), [kv], [100])
    assert e.value.code == avsg.EINVAL                                   # K above max_topk
    pageable = np.zeros(100 * 32, np.uint8)
    with pytest.raises(avsg.AvsgError) as e:
        ctx.step([0], idx, [pageable], [100])                            # host KV that the GPU cannot read
    assert e.value.code == avsg.EINVAL
    with pytest.raises(avsg.AvsgError) as e:
        avsg.Context(1, 64, 32, 40, 2, 4)                                # Eq. 7 at create
    assert e.value.code == avsg.ECAPACITY
    assert ctx.sync_status() == 0


def test_small_context_created_after_a_large_one_does_not_break_it(avsg):
    import torch
    rb = 32
    kv = avsg.pinned_empty(20000 * rb)
    tr.fill_kv(kv.data_ptr(), 5, 0, 20000, rb)
    big = avsg.Context(1, 8192, rb, 2048, 2, 16)
    small = avsg.Context(1, 64, rb, 16, 1, 16)
    Xs = torch.arange(16, dtype=torch.int32, device="cuda").reshape(1, 1, 16)
    small.step([0], Xs, [kv], [20000])
    Xb = torch.arange(4096, dtype=torch.int32, device="cuda").reshape(1, 2, 2048) * 3
    out = big.step([0], Xb, [kv], [20000])                   # must still launch with its large shared memory
    torch.cuda.synchronize()
    assert out.miss_count.cpu().numpy().sum() == 4096 and big.sync_status() == 0


# ---- the direct-address index gives the same results as the shared-memory hash index ---------------------------
@pytest.mark.parametrize("name,kw,every", [
    ("C1", {}, 1), ("C2", {}, 16), ("C3", {}, 32), ("C4", {}, 32), ("C5", {}, 16),
])
def test_direct_index_full(avsg, name, kw, every):
    _parity(tr.workload(name, **kw), index_mode=avsg.INDEX_DIRECT, buffer_every=every)


@pytest.mark.parametrize("name,kw", SHAPES)
def test_direct_index_shapes(avsg, name, kw):
    _parity(tr.workload(name, **kw), index_mode=avsg.INDEX_DIRECT)


def test_direct_index_import_restore_and_bad_ids(avsg):
    import torch
    rb, S, K, ctxlen = 32, 128, 16, 2000
    host = np.empty(ctxlen * rb, np.uint8)
    tr.fill_kv(host, 2, 0, ctxlen, rb)
    dkv = torch.from_numpy(host).cuda()
    ctx = avsg.Context(2, S, rb, K, 1, 4, index_mode=avsg.INDEX_DIRECT, max_context=ctxlen)
    orc = OracleTable(S, rb, 4)
    rng = np.random.default_rng(1)
    sels = [np.sort(rng.choice(ctxlen, K, replace=False)).astype(np.int32) for _ in range(40)]
    for t in range(20):
        ctx.step([0], torch.from_numpy(sels[t][None, None]).cuda(), [dkv], [ctxlen])
        orc.step(sels[t][None], ctxlen, host)
    tok, life = ctx.export_state(0)
    ctx.import_state(1, tok, life)                         # resume into a table whose index has never seen these ids
    ctx.save_state()
    for t in range(20, 30):
        a = ctx.step([1], torch.from_numpy(sels[t][None, None]).cuda(), [dkv], [ctxlen])
        r = orc.step(sels[t][None], ctxlen, host)
        assert (a.slots.cpu().numpy()[0] == r.O).all() and (a.hit.cpu().numpy()[0] == r.M).all()
    first = ctx.export_state(1)
    ctx.restore_state()                                    # back to the snapshot: the same ten steps replay identically
    orc2 = OracleTable(S, rb, 4)
    orc2.import_state(tok, life)
    for t in range(20, 30):
        a = ctx.step([1], torch.from_numpy(sels[t][None, None]).cuda(), [dkv], [ctxlen])
        r = orc2.step(sels[t][None], ctxlen, host)
        assert (a.slots.cpu().numpy()[0] == r.O).all() and (a.hit.cpu().numpy()[0] == r.M).all()
    again = ctx.export_state(1)
    assert (first[0] == again[0]).all() and (first[1] == again[1]).all()
    assert ctx.sync_status() == 0
    bad = np.sort(rng.choice(ctxlen, K, replace=False)).astype(np.int32)
    bad[-1] = ctxlen + 5                                   # an id the direct index cannot hold
    out = ctx.step([0], torch.from_numpy(bad[None, None]).cuda(), [dkv], [ctxlen + 10])
    assert out.slots.cpu().numpy()[0, 0, -1] == -1
    assert ctx.sync_status() != 0                          # reported, not faulted
    with pytest.raises(avsg.AvsgError):
        avsg.Context(1, S, rb, K, 1, 4, index_mode=avsg.INDEX_DIRECT, max_context=0)


@pytest.mark.parametrize("index,cluster,mode", [
    ("INDEX_HASH", 0, "XFER_SM_BALANCED"), ("INDEX_DIRECT", 0, "XFER_SM_OVERLAP"), ("INDEX_PAPER", 0, "XFER_SM_BALANCED"),
    ("INDEX_HASH", 2, "XFER_SM_OVERLAP"), ("INDEX_DIRECT", 4, "XFER_SM_BALANCED"), ("INDEX_HASH", 0, "XFER_ALL_K"),
    ("INDEX_HASH", 0, "XFER_POSITION_LEVEL"),
])
def test_ids_beyond_the_host_rows_are_not_fetched(avsg, index, cluster, mode):
    """With kv_rows stated, an id at or beyond a table's host rows is taken as padding (slot -1, nothing read from
    host memory) and reported in the status word; everything else goes on as if the id had been padding."""
    import torch
    from oracle import LiteralOracleTable
    rb, S, K, rows, n = 48, 256, 24, 3000, 3
    kv = avsg.pinned_empty(rows * rb)                     # exactly `rows` rows: an unchecked id beyond it would read
    tr.fill_kv(kv.data_ptr(), 6, 0, rows, rb)             # outside the allocation
    literal = index == "INDEX_PAPER"
    all_k = mode == "XFER_ALL_K"
    ctx = avsg.Context(n, S, rb, K, 2, 4, index_mode=getattr(avsg, index), max_context=1 << 20,
                       stage_one_cluster=cluster, transfer_mode=getattr(avsg, mode))
    orc = [LiteralOracleTable(S, rb, 4) if literal else OracleTable(S, rb, 4) for _ in range(n)]
    rng = np.random.default_rng(9)
    saw_bad = False
    for t in range(12):
        X = np.stack([np.stack([rng.permutation(rows)[:K] for _ in range(2)]) for _ in range(n)]).astype(np.int32)
        if t % 3 == 1:                                    # some calls carry ids the host KV does not have
            X[0, 0, 3] = rows
            X[1, 1, 7] = rows + 123456
            X[2, 0, 0] = 0x7FFFFFFF
            saw_bad = True
        out = ctx.step(list(range(n)), torch.from_numpy(X).cuda(), [kv] * n, [rows] * n, kv_rows=[rows] * n)
        torch.cuda.synchronize()
        Xo = np.where(X >= rows, -1, X)                   # what the operator must have seen
        for i in range(n):
            if all_k:
                want = orc[i].step_all_k(Xo[i], kv.numpy(), rb)
                assert (out.slots[i].cpu().numpy() == want).all(), (t, i)
                continue
            r = orc[i].step(Xo[i], rows, kv.numpy(), rb)
            assert (out.slots[i].cpu().numpy() == r.O).all() and (out.hit[i].cpu().numpy() == r.M).all(), (t, i)
            assert (out.miss_count[i].cpu().numpy() == r.n).all(), (t, i)
            assert (ctx.buffer(i).cpu().numpy() == orc[i].rows()).all(), (t, i)
        status = ctx.sync_status()
        assert status == (avsg.STATUS_BAD_ID if saw_bad else 0), (t, status)
    ctx.clear_status()
    assert ctx.sync_status() == 0


# ---- degenerate selections --------------------------------------------------------------------------------------
@pytest.mark.parametrize("index_mode", [0, 1])
def test_degenerate_selections(avsg, index_mode):
    import torch
    rb, S, ctxlen = 32, 32, 500
    host = np.empty(ctxlen * rb, np.uint8)
    tr.fill_kv(host, 4, 0, ctxlen, rb)
    kv = avsg.pinned_empty(ctxlen * rb)
    kv.numpy()[:] = host
    rng = np.random.default_rng(index_mode)
    for K, n_q in [(1, 1), (1, 8), (4, 8), (32, 1), (7, 3)]:
        ctx = avsg.Context(1, S, rb, K, n_q, 2, index_mode=index_mode, max_context=ctxlen)
        orc = OracleTable(S, rb, 2)
        for t in range(30):
            X = np.stack([np.sort(rng.choice(ctxlen, K, replace=False)) for _ in range(n_q)]).astype(np.int32)
            if t % 5 == 4:
                X[n_q - 1, :] = -1                                   # a token made of padding only
            if t % 7 == 6 and K > 1:
                X[0, K // 2:] = -1                                   # a half-padded token
            out = ctx.step([0], torch.from_numpy(X[None]).cuda(), [kv], [ctxlen])
            r = orc.step(X, ctxlen, host)
            assert (out.slots.cpu().numpy()[0] == r.O).all(), (K, n_q, t)
            assert (out.hit.cpu().numpy()[0] == r.M).all() and (out.miss_count.cpu().numpy()[0] == r.n).all()
            tok, life = ctx.export_state(0)
            c, l = orc.export_state()
            assert (tok == c).all() and (life == l).all()
        assert (ctx.buffer(0).cpu().numpy() == orc.rows()).all() and ctx.sync_status() == 0


# ---- the paper-literal (lossy) Hash-State mode against its own oracle ---------------------------------------------
def _literal_parity(avsg, w, n_iters=None, R=3, mode=0, permute_seed=None):
    import torch
    from oracle import LiteralOracleTable
    from harness import HostKV
    ids = list(range(w.num_tables))
    traces = {ti: tr.generate(w.tables[ti]) for ti in ids}
    if permute_seed is not None:             # ids in a seeded random order: position order differs from id order
        for ti in ids:
            X, N = traces[ti]
            order = np.argsort(np.random.default_rng([permute_seed, ti]).random(X.shape), axis=-1)
            traces[ti] = (np.ascontiguousarray(np.take_along_axis(X, order, axis=-1)), N)
    kv = HostKV(w, ids)
    ctx = avsg.Context(num_tables=len(ids), buffer_slots=w.buffer_slots, row_bytes=w.row_bytes, max_topk=w.topk,
                       max_tokens=w.n_q, max_lifetime=w.max_lifetime, index_mode=avsg.INDEX_PAPER, probe_retries=R,
                       transfer_mode=mode)
    orc = {ti: LiteralOracleTable(w.buffer_slots, w.row_bytes, w.max_lifetime, R=R) for ti in ids}
    T = w.n_iters if n_iters is None else n_iters
    for t in range(T):
        for grp in w.calls:
            X = np.stack([traces[ti][0][t] for ti in grp])
            vlen = [int(traces[ti][1][t]) for ti in grp]
            out = ctx.step(grp, torch.from_numpy(X).cuda(), [kv.t[ti] for ti in grp], vlen, want_arriving=True)
            torch.cuda.synchronize()
            slots, hit, mc = out.slots.cpu().numpy(), out.hit.cpu().numpy(), out.miss_count.cpu().numpy()
            arr = out.arriving.cpu().numpy()
            for k, ti in enumerate(grp):
                r = orc[ti].step(X[k], vlen[k], kv.np[ti])
                assert (hit[k] == r.M).all(), ("hit mask", ti, t)
                assert (slots[k] == r.O).all(), ("slot table", ti, t)
                assert (arr[k] == r.arriving).all(), ("rows that arrive with this call", ti, t)
                assert (mc[k] == r.n).all(), ("miss counts", ti, t)
                c, q = ctx.export_hash_state(ti)
                oc, oq = orc[ti].export_state()
                assert (c == oc).all() and (q == oq).all(), ("packed state", ti, t)
    for ti in ids:
        assert (ctx.buffer(ti).cpu().numpy() == orc[ti].rows()).all(), ("buffer rows", ti)
    assert ctx.sync_status() == 0
    st = ctx.stats()
    tot = {k: sum(o.counters()[k] for o in orc.values()) for k in ("hits", "misses", "extra_decays")}
    assert st["hits"] == tot["hits"] and st["misses"] == tot["misses"] and st["extra_decays"] == tot["extra_decays"]
    return st


def test_paper_literal_mode_full_c2_and_small_c3(avsg):
    st = _literal_parity(avsg, tr.workload("C2"), n_iters=64)
    assert st["hits"] / (st["hits"] + st["misses"]) < 0.91          # lossy: below the exact index's 92.4 %
    _literal_parity(avsg, tr.workload("C3", requests=6, layers=2, n_iters=10))


def test_paper_literal_mode_with_overlapped_stage_two(avsg):
    _literal_parity(avsg, tr.workload("C2"), n_iters=32, mode=avsg.XFER_SM_OVERLAP)
    _literal_parity(avsg, tr.workload("C3", requests=6, layers=2, n_iters=10), mode=avsg.XFER_SM_OVERLAP)


@pytest.mark.parametrize("kw,R", [
    (dict(topk=37, buffer_slots=128, n_iters=40, context=4096, recent_window=128), 3),
    (dict(topk=16, buffer_slots=32, n_iters=60, context=512, recent_window=64), 1),
    (dict(topk=1000, buffer_slots=2048, n_iters=20, context=65536, recent_window=2048), 7),
    (dict(topk=4096, buffer_slots=8192, n_iters=6, context=65536, recent_window=8192), 3),
])
def test_paper_literal_mode_shapes(avsg, kw, R):
    _literal_parity(avsg, tr.workload("C2", **kw), R=R)


def test_paper_literal_mode_unsorted_ids(avsg):
    # position order decides both the slot of a miss and, in this mode, the winner of a shared bucket
    _literal_parity(avsg, tr.workload("C2", topk=37, buffer_slots=128, n_iters=40, context=4096, recent_window=128),
                    permute_seed=5)
    _literal_parity(avsg, tr.workload("C2", topk=1000, buffer_slots=2048, n_iters=16, context=65536,
                                      recent_window=2048), R=7, permute_seed=6, mode=avsg.XFER_SM_OVERLAP)
    _literal_parity(avsg, tr.workload("C3", requests=4, layers=1, n_iters=8), permute_seed=8)


# ---- randomly drawn shapes: tables, S, K, tokens, L, row size, index and transfer mode -------------------------------
@pytest.mark.parametrize("seed", range(24))
def test_random_shapes(avsg, seed):
    rng = np.random.default_rng(1000 + seed)
    S = int(2 ** rng.integers(5, 14))                                  # 32 .. 8192
    n_q = int(rng.choice([1, 1, 2, 2, 3, 4]))
    k_max = S // n_q
    K = int(rng.integers(1, k_max + 1)) if rng.random() < 0.3 else int(min(k_max, 2 ** rng.integers(0, 12)))
    L = int(rng.choice([1, 2, 8, 16, 30, 31, 64]))
    rb = int(rng.choice([16, 48, 656, 1152]))
    requests = int(rng.choice([1, 2, 5, 9])) if seed < 12 else int(rng.choice([3, 9, 40, 80, 100]))   # 80, 100: rounds
    ctxlen = int(max(2 * K * n_q, rng.integers(K * n_q + 8, 40 * K * n_q + 64)))
    base = rng.choice(["C2", "C4", "C5"])
    kw = dict(topk=K, buffer_slots=S, n_iters=int(rng.integers(3, 14)), max_lifetime=L, row_bytes=rb)
    if base == "C2":
        w = tr.workload("C2", context=ctxlen, recent_window=max(1, ctxlen // 8), **kw)
        if n_q != 2:
            base = "C5"
    if base == "C4":
        w = tr.workload("C4", context=ctxlen, requests=requests, hot_size=min(64, ctxlen // 4),
                        hot_range=max(64, ctxlen // 2), **kw)
        if n_q != 2:
            base = "C5"
    if base == "C5":
        w = tr.workload("C5", requests=requests, ctx_lo=max(4, K // 2), ctx_hi=ctxlen, **kw)
    if w.n_q * w.topk > w.buffer_slots:                                  # the MTP recipes have two tokens
        w = tr.workload("C5", requests=requests, ctx_lo=max(4, K // 2), ctx_hi=ctxlen, **kw)
    mode = getattr(avsg, str(rng.choice(["XFER_SM_BALANCED", "XFER_REQUEST_LEVEL", "XFER_POSITION_LEVEL",
                                         "XFER_SM_OVERLAP"])))
    index_mode = int(rng.choice([avsg.INDEX_HASH, avsg.INDEX_DIRECT]))
    cluster = 0
    if seed >= 12:                                                       # the later seeds also force cluster sizes
        cluster = int(rng.choice([0, 0, 2, 4, 8]))
        if cluster and w.buffer_slots // cluster < 32:
            cluster = 0
        if w.num_tables > 20:                                            # keep the big batches small per table
            w = tr.workload("C5", requests=w.num_tables, ctx_lo=max(4, min(K, 64) // 2), ctx_hi=max(256, 8 * min(K, 64)),
                            topk=min(K, 64), buffer_slots=max(64, min(S, 512)), n_iters=kw["n_iters"], max_lifetime=L,
                            row_bytes=rb)
            if cluster and w.buffer_slots // cluster < 32:
                cluster = 0
    _parity(w, mode=mode, index_mode=index_mode, host_io=bool(rng.random() < 0.3),
            xfer_geometry=(int(rng.choice([1, 37, 148, 300])), int(rng.choice([32, 128, 256, 1024]))),
            permute_seed=seed if seed % 2 else None, cluster=cluster)
