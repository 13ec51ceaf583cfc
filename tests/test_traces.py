"""The seeded input generators: shapes, determinism and the statistics the recipes promise."""
import numpy as np
import pytest

import avsg_traces as tr


@pytest.mark.parametrize("name,kw", [
    ("C1", {}),
    ("C2", dict(n_iters=24)),
    ("C4", dict(n_iters=8, requests=2)),
    ("C5", dict(n_iters=6, requests=4)),
])
def test_selection_is_a_sorted_set_below_the_limit(name, kw):
    w = tr.workload(name, **kw)
    for cfg in w.tables:
        X, N = tr.generate(cfg)
        assert X.shape == (cfg.n_iters, cfg.n_q, cfg.topk) and N.shape == (cfg.n_iters,)
        assert (np.diff(X, axis=2) > 0).all()                      # ascending, hence unique
        assert X.min() >= 0
        for g in range(cfg.n_q):
            lim = N + g if cfg.ctx_growth else N
            assert (X[:, g, :].max(axis=1) < lim).all()
        if cfg.ctx_growth:
            assert (np.diff(N) == cfg.n_q).all() and N[-1] + cfg.n_q == cfg.context
        X2, N2 = tr.generate(cfg)
        assert (X == X2).all() and (N == N2).all()                 # deterministic


def test_overlap_statistics():
    w = tr.workload("C1")
    X, _ = tr.generate(w.tables[0])
    flat = X.reshape(-1, w.topk)
    ov = [len(np.intersect1d(flat[i], flat[i - 1])) for i in range(1, len(flat))]
    assert min(ov) >= int(0.9 * w.topk)                            # keep = floor(0.9 K), plus chance re-draws
    w = tr.workload("C2", n_iters=100)
    X, _ = tr.generate(w.tables[0])
    flat = X.reshape(-1, w.topk)
    ov = np.array([len(np.intersect1d(flat[i], flat[i - 1])) for i in range(1, len(flat))]) / w.topk
    assert abs(ov.mean() - 0.9) < 0.02                             # Beta(18, 2) has mean 0.9


def test_padding_when_context_is_shorter_than_k():
    cfg = tr.TraceConfig(seed=1, table=0, topk=64, n_q=1, n_iters=3, context=40, rho_fixed=0.5)
    X, N = tr.generate(cfg)
    assert (X[:, 0, :40] == np.arange(40)).all() and (X[:, 0, 40:] == -1).all()


def test_tables_have_independent_streams():
    w = tr.workload("C3", n_iters=2, requests=2, layers=2)
    assert w.calls == [[0, 1], [2, 3]]
    a, _ = tr.generate(w.tables[0])
    b, _ = tr.generate(w.tables[1])
    assert (a != b).any()


def test_host_kv_is_a_pure_function_of_position():
    rb = 656
    buf = np.zeros(100 * rb, np.uint8)
    tr.fill_kv(buf, 7, 3, 100, rb)
    rows = tr.kv_rows(7, 3, [0, 17, 99], rb)
    assert (rows == buf.reshape(100, rb)[[0, 17, 99]]).all()
    part = np.zeros(10 * rb, np.uint8)
    tr.fill_kv(part, 7, 3, 10, rb, first_row=40)
    assert (part == buf[40 * rb:50 * rb]).all()
    assert (tr.kv_rows(7, 4, [17], rb) != rows[1]).any()           # another table, other bytes
    assert (tr.kv_rows(7, 3, [17], rb, version=1) != rows[1]).any()
    # strided layout leaves the gap untouched
    wide = np.full(10 * 1024, 0xEE, np.uint8)
    tr.fill_kv(wide, 7, 3, 10, rb, row_stride=1024)
    w2 = wide.reshape(10, 1024)
    assert (w2[:, :rb] == buf.reshape(100, rb)[:10]).all() and (w2[:, rb:] == 0xEE).all()


def test_c5_contexts_are_spread_log_uniformly():
    w = tr.workload("C5")
    ctx = np.array([t.context for t in w.tables])
    assert ctx.min() >= 4096 and ctx.max() <= 524288 and w.num_tables == 64
    assert (ctx < 46341).sum() > 16 and (ctx >= 46341).sum() > 16  # both halves of the log range are populated
    rho = np.array([t.rho_fixed for t in w.tables])
    assert rho.min() >= 0.5 and rho.max() < 0.99
