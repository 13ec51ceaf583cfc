"""avsg_step_noalloc against avsg_step, through the C ABI.

The no-alloc entry point serves callers that cannot allocate device memory at call time: an engine whose
own pool already holds all of it, or a path where the device-wide synchronisation of an allocation is not
acceptable.  The caller owns the table state; the library's scratch is a fixed array in its image.  This
test checks that the entry point gives the same results, bit for bit, as the context-based one, on
several calls in a row (the scratch array keeps the previous call's contents between calls).

This file is collected last on purpose, so that a failure here cannot hide the other tests in a run that
stops at the first failure.
"""
import ctypes

import numpy as np
import pytest

import avsg_traces as tr

pytestmark = pytest.mark.gpu


def _run(avsg, torch, w, n_iters):
    n = w.num_tables
    traces = [tr.generate(c) for c in w.tables]
    kv = []
    for ti, cfg in enumerate(w.tables):
        buf = avsg.pinned_empty(cfg.context * w.row_bytes)
        tr.fill_kv(buf.data_ptr(), w.seed, ti, cfg.context, w.row_bytes)
        kv.append(buf)
    ctx = avsg.Context(n, w.buffer_slots, w.row_bytes, w.topk, w.n_q, w.max_lifetime)
    # caller-owned state of the no-alloc path: empty, dead, zeroed rows
    tok = torch.full((n, w.buffer_slots), -1, dtype=torch.int32, device="cuda")
    life = torch.full((n, w.buffer_slots), -1, dtype=torch.int8, device="cuda")
    rows = torch.zeros((n, w.buffer_slots, w.row_bytes), dtype=torch.uint8, device="cuda")
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for t in range(n_iters):
        X = torch.from_numpy(np.stack([traces[i][0][t] for i in range(n)])).cuda()
        vlen = [int(traces[i][1][t]) for i in range(n)]
        ref = ctx.step(list(range(n)), X, kv, vlen)
        slots = torch.full_like(X, -7)
        hit = torch.full(X.shape, 9, dtype=torch.uint8, device="cuda")
        mc = torch.full((n, w.n_q), -7, dtype=torch.int32, device="cuda")
        avsg.step_noalloc(tok, life, rows, X, kv, vlen, max_lifetime=w.max_lifetime, slots=slots, hit=hit,
                          miss_count=mc, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(slots, ref.slots), ("slots", t)
        assert torch.equal(hit, ref.hit), ("hit", t)
        assert torch.equal(mc, ref.miss_count), ("miss counts", t)
        for i in range(n):
            c, l = ctx.export_state(i)
            assert (tok[i].cpu().numpy() == c).all() and (life[i].cpu().numpy() == l).all(), ("state", t, i)
            assert torch.equal(rows[i], ctx.buffer(i)), ("rows", t, i)
    assert ctx.sync_status() == 0


def test_noalloc_matches_context_path_on_consecutive_calls():
    import torch
    assert torch.cuda.is_available()
    import paper_2609_37538_b200 as avsg
    avsg.load_library()
    # a DSA-shaped case at the headline table size, then a small one with other shapes: the second run
    # starts from a scratch array that still holds the first run's miss lists
    _run(avsg, torch, tr.workload("C3", requests=3, layers=1, n_iters=5, context=32768), 5)
    _run(avsg, torch, tr.workload("C4", topk=100, buffer_slots=256, n_iters=6, context=1 << 14, requests=5,
                                  hot_size=32, hot_range=512, max_lifetime=3), 6)


def test_noalloc_at_its_documented_limits():
    """32 tables x 2 tokens x 2048 ids = 131072 ids on 8192-slot tables: the largest call the fixed scratch takes.
    The first (cold) step writes every entry of the scratch's miss list, the following ones are steady steps."""
    import torch
    import paper_2609_37538_b200 as avsg
    avsg.load_library()
    w = tr.workload("C3", requests=avsg.NOALLOC_MAX_TABLES, layers=1, n_iters=3, context=32768)
    assert w.num_tables * w.n_q * w.topk == avsg.NOALLOC_MAX_IDS and w.buffer_slots == 8192
    _run(avsg, torch, w, 3)


def test_noalloc_checks_ids_against_the_stated_host_rows():
    import torch
    import paper_2609_37538_b200 as avsg
    from oracle import OracleTable
    rb, S, K, rows = 32, 64, 8, 500
    kv = avsg.pinned_empty(rows * rb)
    tr.fill_kv(kv.data_ptr(), 3, 0, rows, rb)
    tok = torch.full((1, S), -1, dtype=torch.int32, device="cuda")
    life = torch.full((1, S), -1, dtype=torch.int8, device="cuda")
    buf = torch.zeros((1, S, rb), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    X = np.array([[[5, 499, 500, 17, 100000, 3, 8, 9]]], dtype=np.int32)
    slots = torch.full((1, 1, K), -7, dtype=torch.int32, device="cuda")
    avsg.step_noalloc(tok, life, buf, torch.from_numpy(X).cuda(), [kv], [rows], max_lifetime=4, slots=slots,
                      status=status, kv_rows=[rows])
    torch.cuda.synchronize()
    orc = OracleTable(S, rb, 4)
    r = orc.step(np.where(X[0] >= rows, -1, X[0]), rows, kv.numpy(), rb)
    assert (slots[0].cpu().numpy() == r.O).all() and (buf[0].cpu().numpy() == orc.rows()).all()
    assert int(status.item()) == avsg.STATUS_BAD_ID


def test_noalloc_rejects_what_the_fixed_scratch_cannot_hold():
    import torch
    import paper_2609_37538_b200 as avsg
    lib = avsg.load_library()
    kv = avsg.pinned_empty(4096 * 32)
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")

    def call(n, n_q, K, S):
        kvs = (ctypes.c_void_p * n)(*[kv.data_ptr()] * n)
        vlen = (ctypes.c_int32 * n)(*[4096] * n)
        a = avsg.AvsgNoAllocArgs()
        a.n, a.n_tokens, a.topk, a.buffer_slots, a.row_bytes, a.max_lifetime = n, n_q, K, S, 32, 16
        p = dummy.data_ptr()
        a.tok = a.life = a.buffer = a.indices = a.slots = p          # never reached: the sizes are refused first
        a.kv_base, a.verified_len = ctypes.addressof(kvs), ctypes.addressof(vlen)
        return lib.avsg_step_noalloc(ctypes.byref(a), None)

    assert call(avsg.NOALLOC_MAX_TABLES + 1, 1, 16, 64) == avsg.EUNSUPPORTED      # too many tables
    assert call(32, 2, 4096, 8192) == avsg.EUNSUPPORTED                            # 262144 ids > 131072
    assert call(1, 1, 16, 16384) == avsg.EUNSUPPORTED                              # table too large
    assert call(1, 2, 40, 64) == avsg.ECAPACITY                                    # Eq. 7
    assert call(1, 1, 16, 100) == avsg.EINVAL                                      # not a power of two
    assert b"not supported" in lib.avsg_strerror(avsg.EUNSUPPORTED)
    torch.cuda.synchronize()
