"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's procedure: each one checks it against
a closed form, a textbook set operation, a special case, a hand-worked example
or an invariant the paper states.
"""
import os

import numpy as np
import pytest

import avsg_traces as tr
from oracle import (ORC_ECAPACITY, OracleError, OracleTable, partition, position_range, requests_of_core,
                    workload)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_example(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            key, *vals = line.split()
            out[key] = np.array([int(v) for v in vals], dtype=np.int64)
    return out


# ----------------------------------------------------------------------------
# hand-worked examples (Algorithm 1: pre-decay, refresh-before-allocate, decay
# loop, ordered assignment of dead slots)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["alloc_example.txt", "refresh_example.txt", "descending_example.txt",
                                  "descending_decay_example.txt"])
def test_hand_worked_example(name):
    ex = _read_example(name)
    S, L, g = int(ex["S"][0]), int(ex["L"][0]), int(ex["g"][0])
    t = OracleTable(S, 16, L)
    t.import_state(ex["c_before"], ex["life_before"])
    o, m, n_g, xfer = t.stage_one_token(g, ex["x"])
    c, life = t.export_state()
    assert m.tolist() == ex["m"].tolist()
    assert o.tolist() == ex["o"].tolist()
    assert n_g == int(ex["n_g"][0])
    assert c.tolist() == ex["c_after"].tolist()
    assert life.tolist() == ex["life_after"].tolist()
    assert t.counters()["extra_decays"] == int(ex["extra_decays"][0])
    # transfer list: the misses in order of position, with their slots
    miss = ex["m"] == 0
    assert xfer[:, 0].tolist() == ex["x"][miss].tolist()
    assert xfer[:, 1].tolist() == ex["o"][miss].tolist()


# ----------------------------------------------------------------------------
# Eq. 1 by brute force on tiny inputs: hit iff the id is among the cached ids
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(6))
def test_membership_bruteforce_tiny(seed):
    rng = np.random.default_rng(seed)
    S, K, L = int(rng.choice([16, 32, 64])), int(rng.choice([4, 8, 16])), int(rng.choice([1, 2, 5]))
    n_q = int(rng.choice([1, 2]))
    if n_q * K > S:
        n_q = 1
    t = OracleTable(S, 8, L)
    universe = 3 * S
    for step in range(40):
        # ids in ascending order on even seeds, in a random order on odd seeds (the input need not be sorted)
        X = np.stack([rng.choice(universe, K, replace=False) for _ in range(n_q)]).astype(np.int32)
        if seed % 2 == 0:
            X.sort(axis=1)
        # token by token, so that "resident" is the table content at the moment the token is
        # processed: an old id may be reclaimed by an earlier token of the same iteration (App. B)
        O = np.empty((n_q, K), np.int32)
        for g in range(n_q):
            resident = set(int(v) for v in t.export_state()[0] if v >= 0)
            o, m, n_g, _ = t.stage_one_token(g, X[g])
            for i in range(K):
                assert bool(m[i]) == (int(X[g, i]) in resident), (step, g, i)
            assert n_g == K - int(m.sum())
            O[g] = o
        t.invalidate(universe)
        c, life = t.export_state()
        # every selected id now sits in the slot the operator reported
        for g in range(n_q):
            assert (c[O[g]] == X[g]).all()


# ----------------------------------------------------------------------------
# special case S = K, one token per step: the buffer holds exactly the previous
# selection, so hits = |sel_t ∩ sel_{t-1}| (the adjacent-step reuse of a
# sort-merge matcher, Sec. 2 / App. C), whatever L is.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L", [1, 2, 16])
def test_s_equals_k_is_adjacent_intersection(L):
    rng = np.random.default_rng(100 + L)
    K = 64
    t = OracleTable(K, 8, L)
    prev = np.array([], dtype=np.int32)
    for step in range(30):
        keep = rng.choice(prev, int(0.7 * len(prev)), replace=False) if len(prev) else prev
        pool = np.setdiff1d(np.arange(1000), keep)
        sel = np.sort(np.concatenate([keep, rng.choice(pool, K - len(keep), replace=False)])).astype(np.int32)
        r = t.step(sel[None, :], 1000)
        assert int(r.M.sum()) == len(np.intersect1d(sel, prev))
        assert int(r.n[0]) == K - len(np.intersect1d(sel, prev))
        c, _ = t.export_state()
        assert sorted(c.tolist()) == sorted(sel.tolist())
        prev = sel


# ----------------------------------------------------------------------------
# special case "no pressure": if all ids ever selected fit and the trace is no
# longer than L + 1 steps, nothing is ever reclaimed: hit iff selected before.
# The first configuration (K=256, S=1024, 16 steps, L=16) is such a trace.
# ----------------------------------------------------------------------------
def test_no_pressure_running_union_c1():
    w = tr.workload("C1")
    X, N = tr.generate(w.tables[0])
    assert len(np.unique(X)) <= w.buffer_slots and X.shape[0] <= w.max_lifetime + 1
    t = OracleTable(w.buffer_slots, 8, w.max_lifetime)
    seen = set()
    for step in range(X.shape[0]):
        r = t.step(X[step], int(N[step]))
        expect = np.array([int(x) in seen for x in X[step, 0]], dtype=np.uint8)
        assert (r.M[0] == expect).all()
        seen |= set(int(x) for x in X[step, 0])
    assert t.counters()["extra_decays"] == 0
    # first-fit in slot order: the ids sit in slots 0.. in order of first appearance
    c, _ = t.export_state()
    first_seen = []
    s2 = set()
    for step in range(X.shape[0]):
        for x in X[step, 0]:
            if int(x) not in s2:
                s2.add(int(x))
                first_seen.append(int(x))
    assert c[: len(first_seen)].tolist() == first_seen
    assert (c[len(first_seen):] == -1).all()


# ----------------------------------------------------------------------------
# cold start and unchanged selection
# ----------------------------------------------------------------------------
def test_cold_start_and_unchanged_selection():
    S, K, L = 64, 16, 4
    t = OracleTable(S, 8, L)
    sel = (np.arange(K, dtype=np.int32) * 7 + 3)[None, :]
    r = t.step(sel, 10_000)
    assert r.M.sum() == 0 and r.n[0] == K
    assert r.O[0].tolist() == list(range(K))          # slots 0..K-1 in order of position
    c0, life0 = t.export_state()
    assert (life0[:K] == L).all() and (life0[K:] == -1).all()
    for _ in range(3 * L):                             # far longer than L: hits keep refreshing
        r = t.step(sel, 10_000)
        assert r.M.all() and r.n[0] == 0 and r.xfer.shape[0] == 0
        assert r.O[0].tolist() == list(range(K))
        c, life = t.export_state()
        assert (c == c0).all() and (life == life0).all()


# ----------------------------------------------------------------------------
# lifetime closed form: an id selected once lives L further pre-decays and is
# reclaimable after more than L of them (Sec. 3.5); dead saturates at -1.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L", [1, 3, 16])
def test_lifetime_closed_form(L):
    S, K = 512, 8
    t = OracleTable(S, 8, L)
    first = np.arange(K, dtype=np.int32)
    t.step(first[None, :], 10**6)
    for k in range(1, L + 2):
        other = (np.arange(K, dtype=np.int32) + 1000 * k)[None, :]   # fresh ids; never-used slots abound
        r = t.step(other, 10**6)
        c, life = t.export_state()
        if k <= L:
            assert (life[:K] == L - k).all() and (c[:K] == first).all(), k
            assert r.O[0].tolist() == list(range(k * K, (k + 1) * K))
        else:
            # after L + 1 pre-decays the first slots are dead and, being the lowest-numbered dead
            # slots, are the ones handed to this step's misses
            assert r.O[0].tolist() == list(range(K)) and (c[:K] == other[0]).all()
    assert t.counters()["extra_decays"] == 0


def test_dead_saturates_at_minus_one():
    S, K, L = 64, 4, 2
    t = OracleTable(S, 8, L)
    sel = np.arange(K, dtype=np.int32)[None, :]
    for _ in range(300):                                             # far beyond the range of a signed byte
        t.step(sel, 10**6)
    _, life = t.export_state()
    assert (life[K:] == -1).all() and (life[:K] == L).all()


# ----------------------------------------------------------------------------
# aging is LRU-like: three disjoint selections cycling through a buffer that
# holds two of them always evict the least recent one, so nothing ever hits
# (textbook LRU under a cyclic scan), while two cycling selections always hit.
# ----------------------------------------------------------------------------
def test_cyclic_scan_behaves_like_lru():
    K, L = 32, 16
    sets = [np.arange(K, dtype=np.int32) + 100 * s for s in range(3)]
    t = OracleTable(2 * K, 8, L)
    for step in range(12):
        sel = sets[step % 3]
        before = set(int(v) for v in t.export_state()[0] if v >= 0)
        r = t.step(sel[None, :], 10**6)
        assert r.M.sum() == 0
        after = set(int(v) for v in t.export_state()[0] if v >= 0)
        if step >= 2:
            lru = set(int(v) for v in sets[(step - 2) % 3])       # least recently selected
            assert before - after == lru
    t2 = OracleTable(2 * K, 8, L)
    for step in range(12):
        r = t2.step(sets[step % 2][None, :], 10**6)
        assert bool(r.M.all()) == (step >= 2)


# ----------------------------------------------------------------------------
# MTP sharing (Sec. 3.6, Alg. 4): later tokens hit the reservations of earlier
# ones; one copy per distinct missing id; with S = N_q K and disjoint
# selections no slot reserved in the iteration is reclaimed (Sec. 3.5 proof).
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L", [1, 2, 16])
def test_mtp_sharing_and_preservation(L):
    rng = np.random.default_rng(7 + L)
    K, n_q = 32, 4
    S = n_q * K
    t = OracleTable(S, 8, L)
    universe = 4000
    for step in range(25):
        if step % 3 == 2:      # disjoint selections: the tight case of Eq. 7
            perm = rng.permutation(universe)[: n_q * K]
            X = np.sort(perm.reshape(n_q, K), axis=1).astype(np.int32)
        else:                  # overlapping selections
            base = rng.choice(universe, K + 8 * n_q, replace=False)
            X = np.stack([np.sort(rng.choice(base, K, replace=False)) for _ in range(n_q)]).astype(np.int32)
        resident = set(int(v) for v in t.export_state()[0] if v >= 0)
        r = t.step(X, universe)
        union = set(int(v) for v in X.ravel())
        # ids that were resident at the start may be reclaimed by an earlier token of the same
        # iteration and fetched again by a later one (App. B), so the number of copies is at
        # least the distinct non-resident ids and at most the distinct ids
        assert len(union - resident) <= r.xfer.shape[0] <= len(union)
        assert r.xfer.shape[0] == int(r.n.sum())
        seen = set()
        for g in range(n_q):
            for i in range(K):
                x = int(X[g, i])
                if x in seen:
                    assert r.M[g, i] == 1           # reserved earlier in this iteration => hit
            seen |= set(int(v) for v in X[g])
        c, life = t.export_state()
        for g in range(n_q):                         # every output slot still holds its id at the end
            assert (c[r.O[g]] == X[g]).all()
            assert (life[r.O[g]] >= 0).all()
        # a slot is the destination of at most one copy per step
        assert len(set(r.xfer[:, 1].tolist())) == r.xfer.shape[0]


def test_arriving_marks_exactly_the_rows_that_were_not_in_the_buffer_before():
    """Sec. 3.6 (a later token can match a slot reserved by an earlier token before its data have arrived) read
    together with Sec. 6 (attention on the hits while the misses load): `arriving` is pinned to what the buffer held
    BEFORE the step, byte for byte - not to the bookkeeping it is computed from."""
    rng = np.random.default_rng(11)
    K, n_q, S, rb, universe = 24, 3, 96, 16, 600
    host = rng.integers(0, 256, (universe, rb), dtype=np.uint8)
    assert len({bytes(r) for r in host}) == universe                 # all rows differ
    t = OracleTable(S, rb, 4)
    in_flight_hits = 0
    for step in range(30):
        base = rng.choice(universe, K + 10, replace=False)
        X = np.stack([rng.permutation(rng.choice(base, K, replace=False)) for _ in range(n_q)]).astype(np.int32)
        X[rng.integers(n_q), rng.integers(K)] = -1                   # one padding position
        before = t.rows().copy()
        r = t.step(X, universe, host.reshape(-1))
        after, F = t.rows(), r.arriving
        if step == 0:
            assert (F == (X >= 0)).all()                             # empty buffer: every row has to come
        for g in range(n_q):
            for i in range(K):
                x, o = int(X[g, i]), int(r.O[g, i])
                if x < 0:
                    assert F[g, i] == 0 and o == -1
                    continue
                assert (after[o] == host[x]).all()                   # at the end of the step the row is there
                if F[g, i]:
                    assert (before[o] != host[x]).any()              # ... and it was not there before
                    if r.M[g, i]:
                        in_flight_hits += 1
                        assert g > 0 and x in X[:g]                  # a hit on an earlier token's reservation
                else:
                    assert r.M[g, i] == 1 and (before[o] == host[x]).all()    # readable before Stage Two
    assert in_flight_hits > 50


def test_mtp_cold_start_counts_union():
    K, n_q, S = 64, 4, 256
    rng = np.random.default_rng(3)
    base = rng.choice(5000, 100, replace=False)
    X = np.stack([np.sort(rng.choice(base, K, replace=False)) for _ in range(n_q)]).astype(np.int32)
    t = OracleTable(S, 8, 16)
    r = t.step(X, 5000)
    assert r.M[0].sum() == 0                                        # the first token still misses
    assert r.xfer.shape[0] == len(np.unique(X))                     # one copy per distinct id
    # independent buffers (one table per token) give zero reuse (Table 1, MTP cold start)
    for g in range(n_q):
        ti = OracleTable(S, 8, 16)
        assert ti.step(X[g][None, :], 5000).M.sum() == 0


# ----------------------------------------------------------------------------
# speculative invalidation (Alg. 4 end of step): ids >= N are forgotten, so a
# regenerated host row is fetched again; lifetimes are not touched.
# ----------------------------------------------------------------------------
def test_invalidation_forces_refetch():
    S, K, rb = 32, 4, 16
    N = 100
    kv = np.zeros((N + 4) * rb, np.uint8)
    tr.fill_kv(kv, 1, 0, N + 4, rb)
    t = OracleTable(S, rb, 16)
    X = np.array([[5, 50, 99, 100]], dtype=np.int32)        # id 100 is speculative (>= N)
    r = t.step(X, N, kv)
    c, life = t.export_state()
    assert c[r.O[0, 3]] == -1 and (c[r.O[0, :3]] == X[0, :3]).all()
    assert life[r.O[0, 3]] == 16                             # lifetime untouched
    assert (t.rows()[r.O[0, 3]] == kv[100 * rb:101 * rb]).all()
    tr.fill_kv(kv[100 * rb:], 1, 0, 1, rb, first_row=100, version=1)   # host regenerates row 100
    r2 = t.step(X, N + 1, kv)
    assert r2.M[0].tolist() == [1, 1, 1, 0]                  # must miss although the id is unchanged
    assert (t.rows()[r2.O[0, 3]] == kv[100 * rb:101 * rb]).all()
    assert r2.O[0, 3] != r.O[0, 3]                           # old slot is still alive, so a new one is taken


# ----------------------------------------------------------------------------
# capacity bound Eq. 7 and padding
# ----------------------------------------------------------------------------
def test_capacity_violation_is_reported():
    t = OracleTable(16, 8, 4)
    X = np.arange(24, dtype=np.int32).reshape(2, 12)
    with pytest.raises(OracleError) as ei:
        t.step(X, 100)
    assert ei.value.code == ORC_ECAPACITY


def test_padding_is_neither_hit_nor_miss():
    t = OracleTable(16, 8, 4)
    X = np.array([[3, 9, -1, -1]], dtype=np.int32)
    r = t.step(X, 100)
    assert r.O[0].tolist() == [0, 1, -1, -1] and r.n[0] == 2 and r.M[0].tolist() == [0, 0, 0, 0]
    r = t.step(X, 100)
    assert r.O[0].tolist() == [0, 1, -1, -1] and r.n[0] == 0 and r.M[0].tolist() == [1, 1, 0, 0]
    assert t.counters()["hits"] == 2 and t.counters()["misses"] == 2


# ----------------------------------------------------------------------------
# invariants on DSA-shaped traces (scaled-down versions of the configurations)
# ----------------------------------------------------------------------------
SMALL = [
    ("C2", dict(topk=128, buffer_slots=512, n_iters=40, context=8192, recent_window=256)),
    ("C2", dict(topk=128, buffer_slots=256, n_iters=40, context=8192, recent_window=256)),   # S = N_q K
    ("C4", dict(topk=64, buffer_slots=256, n_iters=30, context=1 << 14, requests=2, hot_size=32, hot_range=512)),
    ("C5", dict(topk=128, buffer_slots=512, n_iters=12, requests=3, ctx_lo=256, ctx_hi=4096)),
]


@pytest.mark.parametrize("name,kw", SMALL)
def test_invariants_on_shaped_traces(name, kw):
    w = tr.workload(name, **kw)
    rb = 16
    for ti, cfg in enumerate(w.tables):
        X, N = tr.generate(cfg)
        kv = np.empty(cfg.context * rb, np.uint8)
        tr.fill_kv(kv, w.seed, ti, cfg.context, rb)
        kv2 = kv.reshape(cfg.context, rb)
        t = OracleTable(w.buffer_slots, rb, w.max_lifetime)
        hits = misses = 0
        for step in range(X.shape[0]):
            c0, life0 = t.export_state()
            r = t.step(X[step], int(N[step]), kv)
            c, life = t.export_state()
            valid = X[step] >= 0
            assert int(r.M.sum()) + int(r.n.sum()) == int(valid.sum())
            hits += int(r.M.sum()); misses += int(r.n.sum())
            live = c[c >= 0]
            assert len(np.unique(live)) == len(live)                       # no id in two slots
            assert life.min() >= -1 and life.max() <= w.max_lifetime
            assert (c < N[step]).all()                                     # invalidation
            rows = t.rows()
            slot_of = {}
            for g in range(X.shape[1]):
                xs, os_ = X[step, g][valid[g]], r.O[g][valid[g]]
                assert (r.O[g][~valid[g]] == -1).all()
                assert (rows[os_] == kv2[xs]).all()                        # attention would read the right bytes
                for x, o in zip(xs.tolist(), os_.tolist()):
                    assert slot_of.setdefault(x, o) == o                  # same id, same slot within an iteration
            assert len(set(slot_of.values())) == len(slot_of)              # distinct ids, distinct slots
            assert len(set(r.xfer[:, 1].tolist())) == r.xfer.shape[0]      # no slot is booked twice
            if step == 0:
                assert r.M[0].sum() == 0                                   # first token of a cold table
        cnt = t.counters()
        assert cnt["hits"] == hits and cnt["misses"] == misses and cnt["rows_copied"] == misses


# ----------------------------------------------------------------------------
# Eq. 6 (balanced partition) and Eq. 13 (request-level assignment)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("n_miss,C", [(0, 7), (1, 148), (147, 148), (148, 148), (149, 148), (9613, 148),
                                      (131072, 148), (5, 1), (1000, 3)])
def test_partition_balanced(n_miss, C):
    ranges = [partition(n_miss, C, c) for c in range(C)]
    sizes = [e - b for b, e in ranges]
    assert ranges[0][0] == 0 and ranges[-1][1] == n_miss
    assert all(ranges[i][1] == ranges[i + 1][0] for i in range(C - 1))     # consecutive, cover once
    assert set(sizes) <= {n_miss // C, -(-n_miss // C)}
    assert max(sizes) - min(sizes) <= 1


@pytest.mark.parametrize("B,C", [(1, 148), (32, 148), (150, 148), (64, 24)])
def test_request_level_assignment(B, C):
    per = [requests_of_core(B, C, c) for c in range(C)]
    assert sum(per) == B and max(per) - min(per) <= 1
    assert per == sorted(per, reverse=True)


# ----------------------------------------------------------------------------
# transfer-all-K comparator: identity slot table, all rows moved
# ----------------------------------------------------------------------------
def test_all_k_comparator():
    rb = 16
    kv = np.empty(500 * rb, np.uint8)
    tr.fill_kv(kv, 9, 0, 500, rb)
    t = OracleTable(64, rb, 16)
    X = np.sort(np.random.default_rng(0).choice(500, (2, 32), replace=True), axis=1).astype(np.int32)
    O = t.step_all_k(X, kv)
    assert O.ravel().tolist() == list(range(64))
    assert (t.rows() == kv.reshape(500, rb)[X.ravel()]).all()
    assert t.counters()["rows_copied"] == 64
    # padding (negative ids) moves nothing and gets no slot; the other positions keep their slots g*K + i
    t2 = OracleTable(64, rb, 16)
    Xp = X.copy()
    Xp[0, 5] = Xp[1, 31] = -1
    O2 = t2.step_all_k(Xp, kv)
    want = np.arange(64)
    want[[5, 63]] = -1
    assert O2.ravel().tolist() == want.tolist()
    assert t2.counters()["rows_copied"] == 62
    keep = want >= 0
    assert (t2.rows()[keep] == kv.reshape(500, rb)[Xp.ravel()[keep]]).all()
    assert not t2.rows()[~keep].any()                      # the two padded slots were never written


# ----------------------------------------------------------------------------
# A request that ends leaves its table as a new request finds it (App. E: every request starts with an empty
# cache): after a busy trace, reset() must give a table that cannot be told from a fresh one - ids, lifetimes,
# rows and all six counters - now and on the steps that follow.
# ----------------------------------------------------------------------------
def test_reset_equals_fresh_table():
    w = tr.workload("C2", topk=64, buffer_slots=128, n_iters=30, context=4096, recent_window=256, max_lifetime=16)
    X, N = tr.generate(w.tables[0])
    rb = 16
    kv = np.empty(w.tables[0].context * rb, np.uint8)
    tr.fill_kv(kv, w.seed, 0, w.tables[0].context, rb)
    used, fresh = OracleTable(w.buffer_slots, rb, w.max_lifetime), OracleTable(w.buffer_slots, rb, w.max_lifetime)
    for t in range(20):
        used.step(X[t], int(N[t]), kv)
    c = used.counters()
    assert c["misses"] > 0 and c["extra_decays"] > 0 and used.rows().any()       # the trace was busy
    used.reset()
    assert used.counters() == fresh.counters() == dict.fromkeys(c, 0)
    assert (used.export_state()[0] == -1).all() and (used.export_state()[1] == -1).all()
    assert not used.rows().any()
    for t in range(20, 30):                                                      # and behaves like one from here on
        a, b = used.step(X[t], int(N[t]), kv), fresh.step(X[t], int(N[t]), kv)
        assert (a.O == b.O).all() and (a.M == b.M).all() and (a.n == b.n).all()
    assert used.counters() == fresh.counters()
    assert (used.rows() == fresh.rows()).all()


# ----------------------------------------------------------------------------
# Host rows with a stride: row x starts at x * row_stride and only its first row_bytes bytes are the row.  A
# padded host array (gaps filled with 0xEE) must give exactly the rows of the packed array, for the operator
# and for the transfer-all-K comparator.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("stride", [48, 1024])
def test_strided_host_rows_equal_packed_rows(stride):
    rb, ctx_len = 32, 2048
    w = tr.workload("C2", topk=48, buffer_slots=128, n_iters=12, context=ctx_len, recent_window=256, row_bytes=rb)
    X, N = tr.generate(w.tables[0])
    packed = np.empty(ctx_len * rb, np.uint8)
    tr.fill_kv(packed, w.seed, 0, ctx_len, rb)
    padded = np.full(ctx_len * stride, 0xEE, np.uint8)
    padded.reshape(ctx_len, stride)[:, :rb] = packed.reshape(ctx_len, rb)
    a, b = OracleTable(w.buffer_slots, rb, 4), OracleTable(w.buffer_slots, rb, 4)
    for t in range(X.shape[0]):
        ra, rb_ = a.step(X[t], int(N[t]), packed), b.step(X[t], int(N[t]), padded, stride)
        assert (ra.O == rb_.O).all() and (ra.xfer == rb_.xfer).all()
        assert (a.rows() == b.rows()).all(), t
        # and the rows are the right ones: slot O[g, i] holds host row X[g, i]
        for g in range(X.shape[1]):
            assert (b.rows()[rb_.O[g]] == packed.reshape(ctx_len, rb)[X[t, g]]).all()
    assert a.counters() == b.counters()
    ka, kb = OracleTable(w.buffer_slots, rb, 4), OracleTable(w.buffer_slots, rb, 4)
    ka.step_all_k(X[3], packed)
    kb.step_all_k(X[3], padded, stride)
    assert (ka.rows() == kb.rows()).all() and ka.rows().any()
    assert (kb.rows()[: X[3].size] == packed.reshape(ctx_len, rb)[X[3].ravel()]).all()


# ----------------------------------------------------------------------------
# Eq. 14 / Eq. 15: equal top-K position partitioning covers every position once, sizes differ by at most
# one, and the work of a core is the number of misses in its range - so two cores with equal shares of
# positions can have very different work, down to none at all for an all-hit range.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("P,C", [(2048, 148), (65536, 148), (100, 7), (5, 8)])
def test_position_partition(P, C):
    ranges = [position_range(P, C, c) for c in range(C)]
    assert ranges[0][0] == 0 and ranges[-1][1] == P
    assert all(ranges[i][1] == ranges[i + 1][0] for i in range(C - 1))
    sizes = [e - b for b, e in ranges]
    assert max(sizes) - min(sizes) <= 1
    assert [b for b, _ in ranges] == [c * P // C for c in range(C)]            # the floor formula itself


def test_position_partition_work_is_hit_dependent():
    K, C = 64, 4
    X = np.arange(K, dtype=np.int32)
    M = np.zeros(K, np.uint8)
    M[:16] = 1                                      # the first core's whole range hits
    work = [workload(M, X, *position_range(K, C, c)) for c in range(C)]
    assert work == [0, 16, 16, 16] and sum(work) == int((1 - M).sum())
    # Eq. 15: W_c - W_d = hits(d) - hits(c) for equal-sized ranges
    hits = [int(M[slice(*position_range(K, C, c))].sum()) for c in range(C)]
    assert all(work[c] - work[d] == hits[d] - hits[c] for c in range(C) for d in range(C))
    Xp = X.copy(); Xp[60:] = -1                     # padding is neither work nor a hit
    assert workload(M, Xp, *position_range(K, C, 3)) == 12
