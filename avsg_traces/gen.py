"""ctypes binding of the trace / host-KV generator and the five workload recipes.

The recipes follow the shapes of DSA decoding the operator is evaluated on:
top-K = 2048 ids per query token out of a 128 Ki .. 1 Mi context, an
8192-slot device buffer, 656-byte KV rows (512 B fp8 latent + 16 B scales +
128 B rope, opaque bytes here), and 2 query tokens per iteration when
multi-token prediction is on.  They stand in for production traces, which are
not available; only their statistics (overlap between consecutive selections,
recency bias, hot positions) are imitated.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tracegen.c")
_LIB = os.path.join(_HERE, "libtracegen.so")


def build_library(force: bool = False) -> str:
    """Compiles tracegen.c into libtracegen.so next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _TgConfig(ctypes.Structure):
    _fields_ = [
        ("seed", ctypes.c_uint64),
        ("table", ctypes.c_uint32),
        ("topk", ctypes.c_uint32),
        ("n_q", ctypes.c_uint32),
        ("n_iters", ctypes.c_uint32),
        ("context", ctypes.c_int64),
        ("ctx_growth", ctypes.c_int32),
        ("rho_kind", ctypes.c_int32),
        ("rho_fixed", ctypes.c_double),
        ("beta_a", ctypes.c_int32),
        ("beta_b", ctypes.c_int32),
        ("p_recent", ctypes.c_double),
        ("recent_window", ctypes.c_uint32),
        ("p_hot", ctypes.c_double),
        ("hot_size", ctypes.c_uint32),
        ("hot_range", ctypes.c_uint32),
        ("p_hist", ctypes.c_double),
        ("hist_sigma", ctypes.c_double),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_library())
        lib.tg_generate.argtypes = [ctypes.POINTER(_TgConfig), ctypes.c_void_p, ctypes.c_void_p]
        lib.tg_generate.restype = ctypes.c_int
        lib.tg_fill_kv.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64,
                                   ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32]
        lib.tg_fill_kv.restype = None
        lib.tg_kv_rows.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p,
                                   ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32]
        lib.tg_kv_rows.restype = None
        lib.tg_log_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int64, ctypes.c_int64]
        lib.tg_log_uniform.restype = ctypes.c_int64
        lib.tg_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_double, ctypes.c_double]
        lib.tg_uniform.restype = ctypes.c_double
        _lib = lib
    return _lib


@dataclass(frozen=True)
class TraceConfig:
    """Recipe of one table's trace (mirrors the C struct)."""
    seed: int
    table: int
    topk: int
    n_q: int
    n_iters: int
    context: int
    ctx_growth: bool = False
    rho_fixed: Optional[float] = None       # fixed overlap, or
    beta: Optional[Tuple[int, int]] = None  # Beta(a, b) overlap with integer a, b
    p_recent: float = 0.0
    recent_window: int = 0
    p_hot: float = 0.0
    hot_size: int = 0
    hot_range: int = 0
    p_hist: float = 0.0          # share of new ids re-drawn from earlier selections ("historical recall")
    hist_sigma: float = 0.0      # per-token jitter of p_hist (normal, clipped to [0, 1])

    def _c(self) -> _TgConfig:
        c = _TgConfig()
        c.seed, c.table, c.topk, c.n_q, c.n_iters = self.seed, self.table, self.topk, self.n_q, self.n_iters
        c.context, c.ctx_growth = self.context, int(self.ctx_growth)
        if self.beta is not None:
            c.rho_kind, c.beta_a, c.beta_b, c.rho_fixed = 1, self.beta[0], self.beta[1], 0.0
        else:
            c.rho_kind, c.beta_a, c.beta_b = 0, 1, 1
            c.rho_fixed = 0.0 if self.rho_fixed is None else float(self.rho_fixed)
        c.p_recent, c.recent_window = self.p_recent, self.recent_window
        c.p_hot, c.hot_size, c.hot_range = self.p_hot, self.hot_size, self.hot_range
        c.p_hist, c.hist_sigma = self.p_hist, self.hist_sigma
        return c


def generate(cfg: TraceConfig) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (X[T, N_q, K] int32 ascending with -1 padding, verified_len[T] int32)."""
    X = np.empty((cfg.n_iters, cfg.n_q, cfg.topk), dtype=np.int32)
    N = np.empty((cfg.n_iters,), dtype=np.int32)
    c = cfg._c()
    rc = _load().tg_generate(ctypes.byref(c), X.ctypes.data, N.ctypes.data)
    if rc != 0:
        raise ValueError("bad trace configuration: %r" % (cfg,))
    return X, N


def fill_kv(dst, seed: int, table: int, n_rows: int, row_bytes: int, *, first_row: int = 0,
            row_stride: Optional[int] = None, version: int = 0) -> None:
    """Fills rows [first_row, first_row+n_rows) of a table's host KV.

    dst: writable uint8 numpy array, or an integer address, pointing at the first of those rows.
    """
    if row_bytes % 8:
        raise ValueError("row_bytes must be a multiple of 8")
    stride = row_bytes if row_stride is None else row_stride
    if isinstance(dst, np.ndarray):
        assert dst.dtype == np.uint8 and dst.flags.c_contiguous
        assert dst.size >= (n_rows - 1) * stride + row_bytes if n_rows else True
        addr = dst.ctypes.data
    else:
        addr = int(dst)
    _load().tg_fill_kv(addr, seed, table, first_row, n_rows, row_bytes, stride, version)


def kv_rows(seed: int, table: int, rows: Sequence[int], row_bytes: int, version: int = 0) -> np.ndarray:
    """Recomputes the given rows of a table's host KV: uint8 [len(rows), row_bytes]."""
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    out = np.empty((r.size, row_bytes), dtype=np.uint8)
    _load().tg_kv_rows(out.ctypes.data, seed, table, r.ctypes.data, r.size, row_bytes, version)
    return out


@dataclass
class Workload:
    """One evaluation configuration: a set of tables and how calls group them."""
    name: str
    seed: int
    buffer_slots: int            # S
    row_bytes: int
    max_lifetime: int            # L
    topk: int                    # K
    n_q: int                     # N_q
    n_iters: int                 # T
    tables: List[TraceConfig] = field(default_factory=list)
    calls: List[List[int]] = field(default_factory=list)   # table ids per operator call, per iteration
    note: str = ""

    @property
    def num_tables(self) -> int:
        return len(self.tables)

    def host_kv_bytes(self) -> int:
        return sum(t.context for t in self.tables) * self.row_bytes

    def traces(self, tables: Optional[Sequence[int]] = None):
        """Generates (X, verified_len) for the given table ids (default: all)."""
        ids = range(self.num_tables) if tables is None else tables
        return {i: generate(self.tables[i]) for i in ids}


ROW_BYTES = 656


def _c1(seed=0, **kw) -> Workload:
    K, S, T = kw.get("topk", 256), kw.get("buffer_slots", 1024), kw.get("n_iters", 16)
    ctx = kw.get("context", 8192)
    t = TraceConfig(seed=seed, table=0, topk=K, n_q=1, n_iters=T, context=ctx, rho_fixed=0.9)
    return Workload("C1", seed, S, ROW_BYTES, 16, K, 1, T, [t], [[0]],
                    "1 table, fixed 90% overlap, uniform new ids")


def _mtp_tables(seed, n_tables, K, T, ctx, beta, n_q=2, **mix) -> List[TraceConfig]:
    return [TraceConfig(seed=seed, table=i, topk=K, n_q=n_q, n_iters=T, context=ctx, ctx_growth=True,
                        beta=beta, **mix) for i in range(n_tables)]


def _c2(seed=2, **kw) -> Workload:
    K, S, T = kw.get("topk", 2048), kw.get("buffer_slots", 8192), kw.get("n_iters", 128)
    ctx = kw.get("context", 131072)
    n_q = kw.get("n_q", 2)
    tabs = _mtp_tables(seed, 1, K, T, ctx, (18, 2), n_q=n_q, p_recent=0.5, recent_window=kw.get("recent_window", 4096))
    return Workload("C2", seed, S, ROW_BYTES, 16, K, n_q, T, tabs, [[0]],
                    "1 table, MTP %d tokens, Beta(18,2) overlap, half recent / half uniform" % n_q)


def _c3(seed=3, **kw) -> Workload:
    K, S, T = kw.get("topk", 2048), kw.get("buffer_slots", 8192), kw.get("n_iters", 64)
    ctx = kw.get("context", 131072)
    n_req, n_layers, n_q = kw.get("requests", 32), kw.get("layers", 4), kw.get("n_q", 2)
    tabs = _mtp_tables(seed, n_req * n_layers, K, T, ctx, (18, 2), n_q=n_q, p_recent=0.5,
                       recent_window=kw.get("recent_window", 4096))
    calls = [[layer * n_req + r for r in range(n_req)] for layer in range(n_layers)]
    return Workload("C3", seed, S, ROW_BYTES, 16, K, n_q, T, tabs, calls,
                    "%d requests x %d layers, one call per layer" % (n_req, n_layers))


def _c4(seed=4, **kw) -> Workload:
    K, S, T = kw.get("topk", 2048), kw.get("buffer_slots", 8192), kw.get("n_iters", 64)
    ctx = kw.get("context", 1 << 20)
    n_req, n_q = kw.get("requests", 16), kw.get("n_q", 2)
    tabs = _mtp_tables(seed, n_req, K, T, ctx, (9, 1), n_q=n_q, p_hot=0.2, hot_size=kw.get("hot_size", 512),
                       hot_range=kw.get("hot_range", 8192))
    return Workload("C4", seed, S, ROW_BYTES, 16, K, n_q, T, tabs, [list(range(n_req))],
                    "%d requests, 1 Mi context, Beta(9,1) overlap, 20%% hot set" % n_req)


def _c5(seed=5, **kw) -> Workload:
    K, S, T = kw.get("topk", 2048), kw.get("buffer_slots", 8192), kw.get("n_iters", 33)
    n_req = kw.get("requests", 64)
    lo, hi = kw.get("ctx_lo", 4096), kw.get("ctx_hi", 524288)
    lib = _load()
    tabs = []
    for i in range(n_req):
        ctx = int(lib.tg_log_uniform(seed, i, lo, hi))
        rho = float(lib.tg_uniform(seed, i, 0.5, 0.99))
        tabs.append(TraceConfig(seed=seed, table=i, topk=K, n_q=1, n_iters=T, context=ctx, rho_fixed=rho))
    return Workload("C5", seed, S, ROW_BYTES, 16, K, 1, T, tabs, [list(range(n_req))],
                    "%d requests, log-uniform contexts, per-request fixed overlap, cold first step" % n_req)


WORKLOADS = {"C1": _c1, "C2": _c2, "C3": _c3, "C4": _c4, "C5": _c5}


def workload(name: str, **overrides) -> Workload:
    """Returns one of the five configurations; keyword overrides shrink it for tests
    (topk, buffer_slots, n_iters, context, requests, layers, ...)."""
    w = WORKLOADS[name](**overrides)
    if "max_lifetime" in overrides:
        w = replace(w, max_lifetime=overrides["max_lifetime"])
    if "row_bytes" in overrides:
        w = replace(w, row_bytes=overrides["row_bytes"])
    return w
