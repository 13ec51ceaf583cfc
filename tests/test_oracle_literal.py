"""The paper-literal (lossy) Hash-State mode of the oracle: hand-worked example, agreement with the exact oracle
when nothing is lost, and the invariants the paper states for it."""
import os

import numpy as np
import pytest

import avsg_traces as tr
from oracle import LITERAL_A1, LiteralOracleTable, OracleTable

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].strip()
        if line:
            k, *v = line.split()
            out[k] = np.array([int(t) for t in v], dtype=np.int64)
    return out


def test_hand_worked_literal_example():
    ex = _read("literal_example.txt")
    S, m = int(ex["S"][0]), 3
    t = LiteralOracleTable(S, 8, int(ex["L"][0]), R=int(ex["R"][0]), a1=int(ex["a1"][0]), a2=int(ex["a2"][0]))
    x = ex["x"].astype(np.int32)[None, :]
    r = t.step(x, 1000)
    c, q = t.export_state()
    assert r.M[0].tolist() == ex["m1"].tolist() and r.O[0].tolist() == ex["o1"].tolist()
    assert c.tolist() == ex["c1"].tolist() and t.lifetimes().tolist() == ex["life1"].tolist()
    assert int(q[3]) & (S - 1) == ex["bucket3_slot1"][0] and (int(q[3]) >> m) & ((1 << 20) - 1) == ex["bucket3_fp1"][0]
    assert (int(q[3]) >> 23) & 1 == 0 and (int(q[0]) >> 23) & 1 == 1          # bucket 3 valid, bucket 0 still invalid
    r = t.step(x, 1000)
    c, q = t.export_state()
    assert r.M[0].tolist() == ex["m2"].tolist() and r.O[0].tolist() == ex["o2"].tolist()
    assert c.tolist() == ex["c2"].tolist() and t.lifetimes().tolist() == ex["life2"].tolist()
    assert int(q[0]) & (S - 1) == ex["bucket0_slot2"][0] and (int(q[0]) >> m) & ((1 << 20) - 1) == ex["bucket0_fp2"][0]
    assert r.xfer.tolist() == [[9, 3]]                                          # the resident id is fetched again


def _reclaim_cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "literal_reclaim_examples.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        key, *vals = line.split()
        if key == "case":
            cur = {"name": vals[0], "steps": [], "buckets": []}
            cases.append(cur)
        elif key == "step":
            cur["steps"].append([int(v) for v in vals])
        elif key == "bucket":
            cur["buckets"].append([int(v) for v in vals])
        else:
            cur[key] = [int(v) for v in vals]
    return cases


@pytest.mark.parametrize("case", _reclaim_cases(), ids=lambda c: c["name"])
def test_hand_worked_reclamation_conditions(case):
    S, m = 8, 3
    t = LiteralOracleTable(S, 8, case["L"][0], R=1, a1=3, a2=5)
    for ids in case["steps"]:
        r = t.step(np.array(ids, dtype=np.int32)[None, :], 1000)
    assert r.M[0].tolist() == case["expect_M"] and r.O[0].tolist() == case["expect_O"]
    assert t.counters()["lost_mappings"] == case["expect_lost"][0]
    _, q = t.export_state()
    for h, slot, fp, invalid in case["buckets"]:
        word = int(q[h])
        assert (word & (S - 1), (word >> m) & ((1 << 20) - 1), (word >> 23) & 1) == (slot, fp, invalid), (h, hex(word))


@pytest.mark.parametrize("seed", range(4))
def test_literal_equals_exact_when_no_mapping_is_lost(seed):
    # A trace that is loss-free by construction: 60 ids whose FIRST buckets (a1 * x mod S, Eq. 9) are pairwise
    # distinct, in a table that holds them all, over fewer steps than L.  Every bucket word starts invalid, hence
    # reusable (Eq. 4), so every id is linked from its own first bucket when it is installed; no other id ever
    # probes that bucket first, nothing expires and nothing is reclaimed.  The bounded probe then finds exactly
    # what is resident, and both oracles must agree on everything.
    rng = np.random.default_rng(seed)
    S, K, L = 4096, 12, 16
    lit, ex = LiteralOracleTable(S, 8, L), OracleTable(S, 8, L)
    pool, taken = [], set()
    for x in rng.permutation(100000):
        h = (LITERAL_A1 * int(x)) % S
        if h not in taken:
            taken.add(h)
            pool.append(int(x))
        if len(pool) == 60:
            break
    pool = np.array(pool)
    assert len(pool) == 60 and len({(LITERAL_A1 * int(x)) % S for x in pool}) == 60
    for step in range(12):
        X = rng.choice(pool, K, replace=False).astype(np.int32)[None, :]        # any order: not sorted
        a, b = lit.step(X, 10**6), ex.step(X, 10**6)
        c, q = lit.export_state()
        live = c[c >= 0]
        assert lit.counters()["lost_mappings"] == 0 and len(live) == len(np.unique(live))
        assert (a.M == b.M).all() and (a.O == b.O).all() and (a.n == b.n).all()
        assert (c == ex.export_state()[0]).all() and (lit.lifetimes() == ex.export_state()[1]).all()
    assert lit.counters()["hits"] == ex.counters()["hits"] > 0


@pytest.mark.parametrize("kw", [
    dict(topk=128, buffer_slots=512, n_iters=40, context=8192, recent_window=256),
    dict(topk=128, buffer_slots=256, n_iters=40, context=8192, recent_window=256),
])
def test_literal_invariants_and_loss(kw):
    w = tr.workload("C2", **kw)
    X, N = tr.generate(w.tables[0])
    rb = 16
    kv = np.empty(w.tables[0].context * rb, np.uint8)
    tr.fill_kv(kv, w.seed, 0, w.tables[0].context, rb)
    kv2 = kv.reshape(-1, rb)
    lit, ex = LiteralOracleTable(w.buffer_slots, rb, w.max_lifetime), OracleTable(w.buffer_slots, rb, w.max_lifetime)
    for t in range(X.shape[0]):
        c0, _ = lit.export_state()
        r = lit.step(X[t], int(N[t]), kv)
        ex.step(X[t], int(N[t]), kv)
        c, q = lit.export_state()
        life = lit.lifetimes()
        assert int(r.M.sum()) + int(r.n.sum()) == X[t].size
        assert life.min() >= -1 and life.max() <= w.max_lifetime and (c < N[t]).all()
        rows = lit.rows()
        resident = set(c0[c0 >= 0].tolist())
        for g in range(X.shape[1]):
            assert (rows[r.O[g]] == kv2[X[t, g]]).all()                  # attention reads the right bytes
            if g == 0:                                                   # full-id comparison: never a false hit
                assert all(int(x) in resident for x in X[t, g][r.M[g] == 1])
        assert len(set(r.xfer[:, 1].tolist())) == r.xfer.shape[0]        # no slot is booked twice in a step
    cl, ce = lit.counters(), ex.counters()
    assert cl["hits"] <= ce["hits"]                                      # bounded probing can only lose hits here
    assert cl["rows_copied"] == cl["misses"]
