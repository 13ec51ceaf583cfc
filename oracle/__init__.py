"""CPU oracle of the AVSG decode-step operator (test infrastructure only).

Thin ctypes wrapper over avsg_oracle.c.  Only tests, the smoke check and the
benchmark's CPU-baseline leg may use this package; the product never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "avsg_oracle.c")
_LIB = os.path.join(_HERE, "libavsg_oracle.so")

ORC_OK, ORC_EINVAL, ORC_ECAPACITY, ORC_ENOMEM = 0, -1, -2, -3


def build_library(force: bool = False) -> str:
    """Compiles avsg_oracle.c with gcc -O2 (no intrinsics, single-threaded)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    # AVSG_ORACLE_LIB: another build of avsg_oracle.c to load instead (the test that checks that the pins catch
    # deliberately broken copies of the oracle uses it)
    lib = ctypes.CDLL(os.environ.get("AVSG_ORACLE_LIB") or build_library())
    vp, u32, i32, u64 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_int32, ctypes.c_uint64
    lib.orc_create.argtypes, lib.orc_create.restype = [u32, u32, i32], vp
    lib.orc_destroy.argtypes, lib.orc_destroy.restype = [vp], None
    lib.orc_reset.argtypes, lib.orc_reset.restype = [vp], None
    lib.orc_find.argtypes, lib.orc_find.restype = [vp, i32], i32
    lib.orc_collect_dead.argtypes, lib.orc_collect_dead.restype = [vp, vp], u32
    lib.orc_stage_one_token.argtypes = [vp, u32, vp, u32, vp, vp, vp, vp]
    lib.orc_stage_one_token.restype = i32
    lib.orc_stage_two.argtypes, lib.orc_stage_two.restype = [vp, vp, u32, vp, u64], None
    lib.orc_invalidate.argtypes, lib.orc_invalidate.restype = [vp, i32], None
    lib.orc_step.argtypes = [vp, vp, u32, u32, i32, vp, u64, vp, vp, vp, vp, vp]
    lib.orc_step.restype = ctypes.c_int
    lib.orc_step_all_k.argtypes = [vp, vp, u32, u32, vp, u64, vp]
    lib.orc_step_all_k.restype = ctypes.c_int
    lib.orc_partition.argtypes = [u64, u32, u32, vp, vp]
    lib.orc_partition.restype = None
    lib.orc_requests_of_core.argtypes, lib.orc_requests_of_core.restype = [u32, u32, u32], u32
    lib.orc_position_range.argtypes, lib.orc_position_range.restype = [u64, u32, u32, vp, vp], None
    lib.orc_workload.argtypes, lib.orc_workload.restype = [vp, vp, u64, u64], u64
    lib.orc_export.argtypes, lib.orc_export.restype = [vp, vp, vp], None
    lib.orc_import.argtypes, lib.orc_import.restype = [vp, vp, vp], None
    lib.orc_rows.argtypes, lib.orc_rows.restype = [vp], vp
    lib.orc_counters.argtypes, lib.orc_counters.restype = [vp, vp], None
    lib.orc_lit_create.argtypes, lib.orc_lit_create.restype = [u32, u32, i32, u32, u32, u32], vp
    lib.orc_lit_destroy.argtypes, lib.orc_lit_destroy.restype = [vp], None
    lib.orc_lit_step.argtypes = [vp, vp, u32, u32, i32, vp, u64, vp, vp, vp, vp, vp]
    lib.orc_lit_step.restype = ctypes.c_int
    lib.orc_lit_export.argtypes, lib.orc_lit_export.restype = [vp, vp, vp], None
    lib.orc_lit_import.argtypes, lib.orc_lit_import.restype = [vp, vp, vp], None
    lib.orc_lit_rows.argtypes, lib.orc_lit_rows.restype = [vp], vp
    lib.orc_lit_counters.argtypes, lib.orc_lit_counters.restype = [vp, vp], None
    _lib = lib
    return lib


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__("oracle error %d" % code)
        self.code = code


class StepResult:
    """Outputs of one oracle step: O, M [N_q, K]; n [N_q]; transfer list (x, o) [n_list, 2]."""
    __slots__ = ("O", "M", "n", "xfer")

    def __init__(self, O, M, n, xfer):
        self.O, self.M, self.n, self.xfer = O, M, n, xfer

    @property
    def arriving(self) -> np.ndarray:
        """[N_q, K] uint8: 1 where the position's row is written by THIS step's Stage Two, i.e. its slot is the
        destination of an entry of the step's transfer list - the position's own entry if it missed, or that of an
        earlier token of the step whose reservation it hit (Sec. 3.6: a later token can match a slot an earlier token
        reserved before its data have arrived).  0: the row was in the buffer before the step, or padding."""
        return ((self.O >= 0) & np.isin(self.O, self.xfer[:, 1])).astype(np.uint8)


class OracleTable:
    """One request(-layer) table: S slots of (id, lifetime) plus S buffer rows."""

    def __init__(self, S: int, row_bytes: int, L: int = 16):
        self._lib = _load()
        self._h = self._lib.orc_create(S, row_bytes, L)
        if not self._h:
            raise OracleError(ORC_EINVAL)
        self.S, self.row_bytes, self.L = S, row_bytes, L

    def __del__(self):
        if getattr(self, "_h", None):
            self._lib.orc_destroy(self._h)
            self._h = None

    def reset(self) -> None:
        self._lib.orc_reset(self._h)

    def find(self, x: int) -> int:
        return self._lib.orc_find(self._h, int(x))

    def collect_dead(self) -> np.ndarray:
        e = np.empty(self.S, np.int32)
        n = self._lib.orc_collect_dead(self._h, e.ctypes.data)
        return e[:n].copy()

    def step(self, X: np.ndarray, N: int, host_kv: Optional[np.ndarray] = None,
             row_stride: Optional[int] = None) -> StepResult:
        """Algorithm 4 on X[N_q, K]; host_kv is the table's host KV as a flat uint8 array (or None)."""
        X = np.ascontiguousarray(X, dtype=np.int32)
        assert X.ndim == 2
        N_q, K = X.shape
        O = np.empty((N_q, K), np.int32)
        M = np.empty((N_q, K), np.uint8)
        n = np.empty((N_q,), np.int32)
        xfer = np.empty((N_q * K, 2), np.int32)
        n_list = ctypes.c_uint32(0)
        kv_ptr = None
        stride = self.row_bytes if row_stride is None else row_stride
        if host_kv is not None:
            assert host_kv.dtype == np.uint8 and host_kv.flags.c_contiguous
            kv_ptr = host_kv.ctypes.data
        rc = self._lib.orc_step(self._h, X.ctypes.data, N_q, K, int(N), kv_ptr, stride,
                                O.ctypes.data, M.ctypes.data, n.ctypes.data, xfer.ctypes.data,
                                ctypes.byref(n_list))
        if rc != ORC_OK:
            raise OracleError(rc)
        return StepResult(O, M, n, xfer[: n_list.value].copy())

    def step_all_k(self, X: np.ndarray, host_kv: Optional[np.ndarray] = None,
                   row_stride: Optional[int] = None) -> np.ndarray:
        X = np.ascontiguousarray(X, dtype=np.int32)
        N_q, K = X.shape
        O = np.empty((N_q, K), np.int32)
        stride = self.row_bytes if row_stride is None else row_stride
        kv_ptr = host_kv.ctypes.data if host_kv is not None else None
        rc = self._lib.orc_step_all_k(self._h, X.ctypes.data, N_q, K, kv_ptr, stride, O.ctypes.data)
        if rc != ORC_OK:
            raise OracleError(rc)
        return O

    def stage_one_token(self, g: int, x: np.ndarray):
        """Algorithm 1 alone (no copy, no invalidation): returns (o, m, n_g, xfer)."""
        x = np.ascontiguousarray(x, dtype=np.int32)
        K = x.size
        o = np.empty(K, np.int32)
        m = np.empty(K, np.uint8)
        xfer = np.empty((K, 2), np.int32)
        n_list = ctypes.c_uint32(0)
        r = self._lib.orc_stage_one_token(self._h, g, x.ctypes.data, K, o.ctypes.data, m.ctypes.data,
                                          xfer.ctypes.data, ctypes.byref(n_list))
        if r < 0:
            raise OracleError(r)
        return o, m, r, xfer[: n_list.value].copy()

    def invalidate(self, N: int) -> None:
        self._lib.orc_invalidate(self._h, int(N))

    def export_state(self) -> Tuple[np.ndarray, np.ndarray]:
        c = np.empty(self.S, np.int32)
        life = np.empty(self.S, np.int8)
        self._lib.orc_export(self._h, c.ctypes.data, life.ctypes.data)
        return c, life

    def import_state(self, c: np.ndarray, life: np.ndarray) -> None:
        c = np.ascontiguousarray(c, dtype=np.int32)
        life = np.ascontiguousarray(life, dtype=np.int8)
        assert c.size == self.S and life.size == self.S
        self._lib.orc_import(self._h, c.ctypes.data, life.ctypes.data)

    def rows(self) -> np.ndarray:
        """The buffer rows as a uint8 [S, row_bytes] copy."""
        p = self._lib.orc_rows(self._h)
        buf = (ctypes.c_uint8 * (self.S * self.row_bytes)).from_address(p)
        return np.frombuffer(buf, dtype=np.uint8).reshape(self.S, self.row_bytes).copy()

    def counters(self) -> dict:
        out = (ctypes.c_uint64 * 6)()
        self._lib.orc_counters(self._h, out)
        keys = ("steps", "tokens", "hits", "misses", "rows_copied", "extra_decays")
        return dict(zip(keys, (int(v) for v in out)))


def partition(n_miss: int, C: int, c: int) -> Tuple[int, int]:
    """Eq. 6: the [begin, end) range of the miss list that core c copies."""
    b, e = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _load().orc_partition(n_miss, C, c, ctypes.byref(b), ctypes.byref(e))
    return b.value, e.value


def requests_of_core(B: int, C: int, c: int) -> int:
    """Eq. 13: number of requests core c serves under request-level assignment."""
    return _load().orc_requests_of_core(B, C, c)


def position_range(n_positions: int, C: int, c: int) -> Tuple[int, int]:
    """Eq. 14: the [begin, end) range of flattened top-K positions that core c walks (hits included)."""
    b, e = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _load().orc_position_range(n_positions, C, c, ctypes.byref(b), ctypes.byref(e))
    return b.value, e.value


def workload(M: np.ndarray, X: np.ndarray, begin: int, end: int) -> int:
    """Eq. 5: number of rows a core moves for the flattened positions [begin, end)."""
    M = np.ascontiguousarray(M, dtype=np.uint8).ravel()
    X = np.ascontiguousarray(X, dtype=np.int32).ravel()
    return int(_load().orc_workload(M.ctypes.data, X.ctypes.data, begin, end))


LITERAL_A1, LITERAL_A2, LITERAL_R = 1000003, 998244353, 3     # two distinct odd primes; the paper's default retry budget


class LiteralOracleTable:
    """The paper-literal Hash-State table (bounded probing, fingerprints, lossy mappings)."""

    def __init__(self, S: int, row_bytes: int, L: int = 16, R: int = LITERAL_R, a1: int = LITERAL_A1,
                 a2: int = LITERAL_A2):
        self._lib = _load()
        self._h = self._lib.orc_lit_create(S, row_bytes, L, R, a1, a2)
        if not self._h:
            raise OracleError(ORC_EINVAL)
        self.S, self.row_bytes, self.L, self.R, self.a1, self.a2 = S, row_bytes, L, R, a1, a2

    def __del__(self):
        if getattr(self, "_h", None):
            self._lib.orc_lit_destroy(self._h)
            self._h = None

    def step(self, X: np.ndarray, N: int, host_kv: Optional[np.ndarray] = None,
             row_stride: Optional[int] = None) -> StepResult:
        X = np.ascontiguousarray(X, dtype=np.int32)
        N_q, K = X.shape
        O = np.empty((N_q, K), np.int32)
        M = np.empty((N_q, K), np.uint8)
        n = np.empty((N_q,), np.int32)
        xfer = np.empty((N_q * K, 2), np.int32)
        n_list = ctypes.c_uint32(0)
        stride = self.row_bytes if row_stride is None else row_stride
        kv_ptr = host_kv.ctypes.data if host_kv is not None else None
        rc = self._lib.orc_lit_step(self._h, X.ctypes.data, N_q, K, int(N), kv_ptr, stride, O.ctypes.data,
                                    M.ctypes.data, n.ctypes.data, xfer.ctypes.data, ctypes.byref(n_list))
        if rc != ORC_OK:
            raise OracleError(rc)
        return StepResult(O, M, n, xfer[: n_list.value].copy())

    def export_state(self) -> Tuple[np.ndarray, np.ndarray]:
        """(c[S] int32, q[S] uint32 packed words)."""
        c = np.empty(self.S, np.int32)
        q = np.empty(self.S, np.uint32)
        self._lib.orc_lit_export(self._h, c.ctypes.data, q.ctypes.data)
        return c, q

    def import_state(self, c: np.ndarray, q: np.ndarray) -> None:
        c = np.ascontiguousarray(c, dtype=np.int32)
        q = np.ascontiguousarray(q, dtype=np.uint32)
        assert c.size == self.S and q.size == self.S
        self._lib.orc_lit_import(self._h, c.ctypes.data, q.ctypes.data)

    def lifetimes(self) -> np.ndarray:
        return (self.export_state()[1] >> 24).astype(np.uint8).view(np.int8)

    def rows(self) -> np.ndarray:
        p = self._lib.orc_lit_rows(self._h)
        buf = (ctypes.c_uint8 * (self.S * self.row_bytes)).from_address(p)
        return np.frombuffer(buf, dtype=np.uint8).reshape(self.S, self.row_bytes).copy()

    def counters(self) -> dict:
        out = (ctypes.c_uint64 * 7)()
        self._lib.orc_lit_counters(self._h, out)
        keys = ("steps", "tokens", "hits", "misses", "rows_copied", "extra_decays", "lost_mappings")
        return dict(zip(keys, (int(v) for v in out)))
