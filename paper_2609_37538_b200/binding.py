"""Thin ctypes binding of libavsg.so: argument marshalling only.

Every step of the operator runs in the CUDA kernels behind the C ABI
(include/avsg.h).  PyTorch supplies device tensors, pinned host tensors and
streams.  If the library is missing the import of this module still works, but
any use raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Union

import numpy as np

from . import build as _build

OK, EINVAL, ENOMEM, ECUDA, ECAPACITY, EDEVICE_STATUS, EUNSUPPORTED = 0, -1, -2, -3, -4, -5, -6
XFER_SM_BALANCED, XFER_COPY_ENGINE, XFER_REQUEST_LEVEL, XFER_ALL_K, XFER_POSITION_LEVEL, XFER_SM_OVERLAP = 0, 1, 2, 3, 4, 5
INDEX_HASH, INDEX_DIRECT, INDEX_PAPER = 0, 1, 2
STATUS_PROBE_EXHAUSTED, STATUS_NO_DEAD_SLOTS, STATUS_BAD_SLOT, STATUS_BAD_SEGMENT, STATUS_BAD_ID, STATUS_WAIT_TIMEOUT = (
    1, 2, 4, 8, 16, 32)
STATUS_LAUNCH_FAILED = 64

EXPORTS = (
    "avsg_create", "avsg_destroy", "avsg_reset", "avsg_reset_async", "avsg_step", "avsg_step_host", "avsg_buffer", "avsg_stats", "avsg_table_stats",
    "avsg_sync_status", "avsg_export_state", "avsg_import_state", "avsg_save_state", "avsg_restore_state",
    "avsg_set_transfer_mode", "avsg_set_timing", "avsg_set_transfer_geometry", "avsg_strerror",
    "avsg_step_noalloc", "avsg_export_hash_state", "avsg_import_hash_state", "avsg_clear_status",
    "avsg_probe_wait_limit", "avsg_host_kv_alloc", "avsg_host_kv_free",
)


class AvsgConfig(ctypes.Structure):
    _fields_ = [("num_tables", ctypes.c_uint32), ("buffer_slots", ctypes.c_uint32), ("row_bytes", ctypes.c_uint32),
                ("max_topk", ctypes.c_uint32), ("max_tokens", ctypes.c_uint32), ("max_lifetime", ctypes.c_int32),
                ("transfer_mode", ctypes.c_uint32), ("device", ctypes.c_int32), ("index_mode", ctypes.c_uint32),
                ("max_context", ctypes.c_uint32), ("probe_retries", ctypes.c_uint32), ("hash_a1", ctypes.c_uint32),
                ("hash_a2", ctypes.c_uint32), ("stage_one_cluster", ctypes.c_uint32)]


class AvsgStepArgs(ctypes.Structure):
    _fields_ = [("n", ctypes.c_uint32), ("table_ids", ctypes.c_void_p), ("n_tokens", ctypes.c_uint32),
                ("topk", ctypes.c_uint32), ("indices", ctypes.c_void_p), ("kv_base", ctypes.c_void_p),
                ("row_stride", ctypes.c_void_p), ("verified_len", ctypes.c_void_p), ("slots", ctypes.c_void_p),
                ("hit", ctypes.c_void_p), ("miss_count", ctypes.c_void_p), ("verified_len_dev", ctypes.c_void_p),
                ("kv_rows", ctypes.c_void_p), ("stage_one_done", ctypes.c_void_p),
                ("stage_one_done_value", ctypes.c_uint64), ("arriving", ctypes.c_void_p)]


class AvsgStats(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_uint64), ("tokens", ctypes.c_uint64), ("hits", ctypes.c_uint64),
                ("misses", ctypes.c_uint64), ("rows_copied", ctypes.c_uint64), ("bytes_copied", ctypes.c_uint64),
                ("extra_decays", ctypes.c_uint64), ("last_stage_one_us", ctypes.c_float),
                ("last_transfer_us", ctypes.c_float), ("last_rows", ctypes.c_uint64),
                ("last_stage_one_kernel_us", ctypes.c_float), ("last_transfer_kernel_us", ctypes.c_float),
                ("last_transfer_start_us", ctypes.c_float), ("last_copy_start_us", ctypes.c_float),
                ("last_first_row_us", ctypes.c_float), ("last_first_block_done_us", ctypes.c_float),
                ("last_call_kernel_us", ctypes.c_float), ("reserved", ctypes.c_float)]


class AvsgNoAllocArgs(ctypes.Structure):
    _fields_ = [("n", ctypes.c_uint32), ("n_tokens", ctypes.c_uint32), ("topk", ctypes.c_uint32),
                ("buffer_slots", ctypes.c_uint32), ("row_bytes", ctypes.c_uint32), ("max_lifetime", ctypes.c_int32),
                ("tok", ctypes.c_void_p), ("life", ctypes.c_void_p), ("buffer", ctypes.c_void_p),
                ("indices", ctypes.c_void_p), ("kv_base", ctypes.c_void_p), ("row_stride", ctypes.c_void_p),
                ("verified_len", ctypes.c_void_p), ("slots", ctypes.c_void_p), ("hit", ctypes.c_void_p),
                ("miss_count", ctypes.c_void_p), ("status", ctypes.c_void_p), ("kv_rows", ctypes.c_void_p)]


NOALLOC_MAX_TABLES, NOALLOC_MAX_IDS = 32, 131072


class AvsgError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s (code %d)" % (what, code))
        self.code = code


_lib = None


def load_library():
    """Loads libavsg.so (built in-tree by build.build_library); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB):
        raise RuntimeError("libavsg.so is missing: run `python __graft_entry__.py` (needs nvcc) to build it; "
                           "there is no CPU fallback")
    lib = ctypes.CDLL(_build.LIB)
    vp, u32, i32 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_int
    lib.avsg_create.argtypes, lib.avsg_create.restype = [ctypes.POINTER(AvsgConfig), ctypes.POINTER(vp)], i32
    lib.avsg_destroy.argtypes, lib.avsg_destroy.restype = [vp], i32
    lib.avsg_reset.argtypes, lib.avsg_reset.restype = [vp, vp, u32], i32
    lib.avsg_step.argtypes, lib.avsg_step.restype = [vp, ctypes.POINTER(AvsgStepArgs), vp], i32
    lib.avsg_step_host.argtypes, lib.avsg_step_host.restype = [vp, ctypes.POINTER(AvsgStepArgs), vp], i32
    lib.avsg_buffer.argtypes, lib.avsg_buffer.restype = [vp, u32, ctypes.POINTER(vp)], i32
    lib.avsg_stats.argtypes, lib.avsg_stats.restype = [vp, ctypes.POINTER(AvsgStats)], i32
    lib.avsg_table_stats.argtypes, lib.avsg_table_stats.restype = [vp, u32, ctypes.POINTER(AvsgStats)], i32
    lib.avsg_sync_status.argtypes, lib.avsg_sync_status.restype = [vp, ctypes.POINTER(u32)], i32
    lib.avsg_reset_async.argtypes, lib.avsg_reset_async.restype = [vp, vp, u32, vp], i32
    lib.avsg_clear_status.argtypes, lib.avsg_clear_status.restype = [vp], i32
    lib.avsg_probe_wait_limit.argtypes, lib.avsg_probe_wait_limit.restype = [vp, vp], i32
    lib.avsg_export_state.argtypes, lib.avsg_export_state.restype = [vp, u32, vp, vp], i32
    lib.avsg_import_state.argtypes, lib.avsg_import_state.restype = [vp, u32, vp, vp], i32
    lib.avsg_save_state.argtypes, lib.avsg_save_state.restype = [vp, vp], i32
    lib.avsg_restore_state.argtypes, lib.avsg_restore_state.restype = [vp, vp], i32
    lib.avsg_set_transfer_mode.argtypes, lib.avsg_set_transfer_mode.restype = [vp, u32], i32
    lib.avsg_set_timing.argtypes, lib.avsg_set_timing.restype = [vp, i32], i32
    lib.avsg_set_transfer_geometry.argtypes, lib.avsg_set_transfer_geometry.restype = [vp, u32, u32], i32
    lib.avsg_strerror.argtypes, lib.avsg_strerror.restype = [i32], ctypes.c_char_p
    lib.avsg_step_noalloc.argtypes, lib.avsg_step_noalloc.restype = [ctypes.POINTER(AvsgNoAllocArgs), vp], i32
    lib.avsg_export_hash_state.argtypes, lib.avsg_export_hash_state.restype = [vp, u32, vp, vp], i32
    lib.avsg_import_hash_state.argtypes, lib.avsg_import_hash_state.restype = [vp, u32, vp, vp], i32
    lib.avsg_host_kv_alloc.argtypes = [ctypes.c_size_t, u32, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_uint64)]
    lib.avsg_host_kv_alloc.restype = i32
    lib.avsg_host_kv_free.argtypes, lib.avsg_host_kv_free.restype = [vp], i32
    _lib = lib
    return lib


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise AvsgError(rc, "%s: %s" % (what, load_library().avsg_strerror(rc).decode()))


HOST_KV_HUGE_PAGES = 1


class HostKV:
    """A range from avsg_host_kv_alloc: pinned, device-mapped host bytes, zero-filled, touched by the calling thread."""

    def __init__(self, nbytes: int, huge_pages: bool = True):
        ptr, huge = ctypes.c_void_p(), ctypes.c_uint64()
        _check(load_library().avsg_host_kv_alloc(int(nbytes), HOST_KV_HUGE_PAGES if huge_pages else 0,
                                                 ctypes.byref(ptr), ctypes.byref(huge)), "avsg_host_kv_alloc")
        self.ptr, self.nbytes, self.huge_bytes = int(ptr.value), int(nbytes), int(huge.value)
        self.mapped_bytes = -(-int(nbytes) // (2 << 20)) * (2 << 20)           # what the library registered

    def data_ptr(self) -> int:
        return self.ptr

    def numpy(self):
        """The bytes as a numpy view (no copy); dead after free()."""
        return np.ctypeslib.as_array((ctypes.c_uint8 * self.nbytes).from_address(self.ptr))

    def free(self) -> None:
        if self.ptr:
            ptr, self.ptr = self.ptr, 0
            _check(load_library().avsg_host_kv_free(ptr), "avsg_host_kv_free")

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def pinned_empty(nbytes: int, huge_pages: bool = False):
    """Pinned (page-locked, device-mapped) host bytes for a table's host KV: a torch tensor, or with huge_pages a
    HostKV range backed by transparent 2 MiB pages where the kernel grants them (App. G)."""
    if huge_pages:
        return HostKV(nbytes, True)
    import torch
    return torch.empty(int(nbytes), dtype=torch.uint8, pin_memory=True)


def _addr(x) -> int:
    """Address of a torch tensor / numpy array, or an integer address itself."""
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if isinstance(x, np.ndarray):
        return int(x.ctypes.data)
    raise TypeError("expected a tensor, an array or an address, got %r" % type(x))


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


class _DevView:
    """Wraps a raw device pointer so that torch can view it without a copy."""

    def __init__(self, ptr: int, shape, typestr: str, owner):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False),
                                         "version": 3, "strides": None}
        self._owner = owner


class StepOutput:
    __slots__ = ("slots", "hit", "miss_count", "arriving")

    def __init__(self, slots, hit, miss_count, arriving=None):
        self.slots, self.hit, self.miss_count, self.arriving = slots, hit, miss_count, arriving


class PreparedCall:
    """The argument block of one recurring call (same tables, same host KV): built once, re-used per step."""

    def __init__(self, ctx: "Context", table_ids: Sequence[int], kv: Sequence, n_tokens: int, topk: int,
                 row_stride: Optional[Sequence[int]] = None, kv_rows: Optional[Sequence[int]] = None):
        n = len(table_ids)
        assert len(kv) == n
        self.ctx, self.n, self.n_tokens, self.topk = ctx, n, n_tokens, topk
        self._keep = list(kv)
        self._tids = (ctypes.c_uint32 * n)(*[int(t) for t in table_ids])
        self._kv = (ctypes.c_void_p * n)(*[_addr(k) for k in kv])
        self._stride = (ctypes.c_uint64 * n)(*[int(s) for s in row_stride]) if row_stride is not None else None
        self._vlen = (ctypes.c_int32 * n)()
        self._rows = (ctypes.c_uint32 * n)(*[int(r) for r in kv_rows]) if kv_rows is not None else None
        a = AvsgStepArgs()
        a.n, a.n_tokens, a.topk = n, n_tokens, topk
        a.table_ids = ctypes.addressof(self._tids)
        a.kv_base = ctypes.addressof(self._kv)
        a.row_stride = ctypes.addressof(self._stride) if self._stride is not None else None
        a.verified_len = ctypes.addressof(self._vlen)
        a.kv_rows = ctypes.addressof(self._rows) if self._rows is not None else None
        self.args = a

    def run(self, indices, verified_len: Sequence[int], slots, hit=None, miss_count=None, stream=None,
            host: bool = False, stage_one_done=None, arriving=None) -> None:
        """indices / slots / hit / miss_count: tensors (device, or pinned host when host=True) or addresses.
        verified_len: a sequence of n ints, or an int32 CUDA tensor [n] that the kernel reads when it runs
        (what a call captured in a CUDA graph needs when the sequences grow between replays).
        stage_one_done: None or (device int64 tensor or address, value): the word receives the value once the
        slot table, hit mask and miss counts of the whole call are final, while the missed rows still travel.
        arriving: None or a uint8 device tensor like hit: 1 where the row comes with this call's Stage Two."""
        a = self.args
        a.arriving = _addr(arriving) if arriving is not None else None
        if stage_one_done is not None:
            a.stage_one_done, a.stage_one_done_value = _addr(stage_one_done[0]), int(stage_one_done[1])
        else:
            a.stage_one_done, a.stage_one_done_value = None, 0
        if hasattr(verified_len, "data_ptr"):
            a.verified_len_dev = verified_len.data_ptr()
        else:
            a.verified_len_dev = None
            self._vlen[:] = [int(v) for v in verified_len]
        a.indices, a.slots = _addr(indices), _addr(slots)
        a.hit = _addr(hit) if hit is not None else None
        a.miss_count = _addr(miss_count) if miss_count is not None else None
        lib = self.ctx._lib
        fn = lib.avsg_step_host if host else lib.avsg_step
        _check(fn(self.ctx._h, ctypes.byref(a), _stream_handle(stream)), "avsg_step")


class Context:
    """Owns the device state of num_tables tables (see avsg_create)."""

    def __init__(self, num_tables: int, buffer_slots: int, row_bytes: int, max_topk: int, max_tokens: int = 1,
                 max_lifetime: int = 16, transfer_mode: int = XFER_SM_BALANCED, device: int = 0,
                 index_mode: int = INDEX_HASH, max_context: int = 0, probe_retries: int = 0, hash_a1: int = 0,
                 hash_a2: int = 0, stage_one_cluster: int = 0):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        cfg = AvsgConfig(num_tables, buffer_slots, row_bytes, max_topk, max_tokens, max_lifetime, transfer_mode,
                         device, index_mode, max_context, probe_retries, hash_a1, hash_a2, stage_one_cluster)
        _check(self._lib.avsg_create(ctypes.byref(cfg), ctypes.byref(self._h)), "avsg_create")
        self.num_tables, self.S, self.row_bytes = num_tables, buffer_slots, row_bytes
        self.max_topk, self.max_tokens, self.L, self.device = max_topk, max_tokens, max_lifetime, device

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.avsg_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the hot call ---------------------------------------------------------------------------------
    def prepare(self, table_ids, kv, n_tokens: int, topk: int, row_stride=None, kv_rows=None) -> PreparedCall:
        return PreparedCall(self, table_ids, kv, n_tokens, topk, row_stride, kv_rows)

    def step(self, table_ids, indices, kv, verified_len, row_stride=None, want_hit: bool = True,
             want_miss_count: bool = True, stream=None, kv_rows=None, stage_one_done=None,
             want_arriving: bool = False) -> StepOutput:
        """One decode iteration. indices: int32 CUDA tensor [n, n_tokens, topk]. Returns device tensors."""
        import torch
        assert indices.is_cuda and indices.dtype == torch.int32 and indices.is_contiguous() and indices.dim() == 3
        n, n_q, K = indices.shape
        call = PreparedCall(self, table_ids, kv, n_q, K, row_stride, kv_rows)
        slots = torch.empty_like(indices)
        hit = torch.empty(indices.shape, dtype=torch.uint8, device=indices.device) if want_hit else None
        mc = torch.empty((n, n_q), dtype=torch.int32, device=indices.device) if want_miss_count else None
        arriving = torch.empty(indices.shape, dtype=torch.uint8, device=indices.device) if want_arriving else None
        call.run(indices, verified_len, slots, hit, mc, stream, stage_one_done=stage_one_done, arriving=arriving)
        out = StepOutput(slots, hit, mc)
        out.arriving = arriving
        return out

    def step_host(self, table_ids, indices, kv, verified_len, row_stride=None, want_hit: bool = True,
                  want_miss_count: bool = True, stream=None) -> StepOutput:
        """Same with host tensors in and out (pinned for asynchrony); returns pinned host tensors."""
        import torch
        assert not indices.is_cuda and indices.dtype == torch.int32 and indices.is_contiguous() and indices.dim() == 3
        n, n_q, K = indices.shape
        call = PreparedCall(self, table_ids, kv, n_q, K, row_stride)
        slots = torch.empty(indices.shape, dtype=torch.int32, pin_memory=True)
        hit = torch.empty(indices.shape, dtype=torch.uint8, pin_memory=True) if want_hit else None
        mc = torch.empty((n, n_q), dtype=torch.int32, pin_memory=True) if want_miss_count else None
        call.run(indices, verified_len, slots, hit, mc, stream, host=True)
        return StepOutput(slots, hit, mc)

    # -- state ----------------------------------------------------------------------------------------
    def reset(self, table_ids: Sequence[int]) -> None:
        ids = (ctypes.c_uint32 * len(table_ids))(*[int(t) for t in table_ids])
        _check(self._lib.avsg_reset(self._h, ids, len(table_ids)), "avsg_reset")

    def reset_async(self, table_ids: Sequence[int], stream=None) -> None:
        """Stream-ordered reset: nothing waits on the host."""
        ids = (ctypes.c_uint32 * len(table_ids))(*[int(t) for t in table_ids])
        _check(self._lib.avsg_reset_async(self._h, ids, len(table_ids), _stream_handle(stream)), "avsg_reset_async")

    def buffer(self, table_id: int):
        """The table's S rows as a uint8 CUDA tensor [S, row_bytes] (a view, no copy)."""
        import torch
        p = ctypes.c_void_p()
        _check(self._lib.avsg_buffer(self._h, table_id, ctypes.byref(p)), "avsg_buffer")
        return torch.as_tensor(_DevView(p.value, (self.S, self.row_bytes), "|u1", self),
                               device="cuda:%d" % self.device)

    def export_state(self, table_id: int):
        tok = np.empty(self.S, np.int32)
        life = np.empty(self.S, np.int8)
        _check(self._lib.avsg_export_state(self._h, table_id, tok.ctypes.data, life.ctypes.data), "avsg_export_state")
        return tok, life

    def import_state(self, table_id: int, tok, life) -> None:
        tok = np.ascontiguousarray(tok, dtype=np.int32)
        life = np.ascontiguousarray(life, dtype=np.int8)
        assert tok.size == self.S and life.size == self.S
        _check(self._lib.avsg_import_state(self._h, table_id, tok.ctypes.data, life.ctypes.data), "avsg_import_state")

    def export_hash_state(self, table_id: int):
        """Paper-literal mode: (c[S] int32, q[S] uint32 packed words)."""
        c = np.empty(self.S, np.int32)
        q = np.empty(self.S, np.uint32)
        _check(self._lib.avsg_export_hash_state(self._h, table_id, c.ctypes.data, q.ctypes.data),
               "avsg_export_hash_state")
        return c, q

    def import_hash_state(self, table_id: int, c, q) -> None:
        c = np.ascontiguousarray(c, dtype=np.int32)
        q = np.ascontiguousarray(q, dtype=np.uint32)
        assert c.size == self.S and q.size == self.S
        _check(self._lib.avsg_import_hash_state(self._h, table_id, c.ctypes.data, q.ctypes.data),
               "avsg_import_hash_state")

    def save_state(self, stream=None) -> None:
        _check(self._lib.avsg_save_state(self._h, _stream_handle(stream)), "avsg_save_state")

    def restore_state(self, stream=None) -> None:
        _check(self._lib.avsg_restore_state(self._h, _stream_handle(stream)), "avsg_restore_state")

    # -- knobs and counters ---------------------------------------------------------------------------
    def set_transfer_mode(self, mode: int) -> None:
        _check(self._lib.avsg_set_transfer_mode(self._h, mode), "avsg_set_transfer_mode")

    def set_timing(self, enable: bool) -> None:
        _check(self._lib.avsg_set_timing(self._h, int(enable)), "avsg_set_timing")

    def set_transfer_geometry(self, blocks: int, threads: int) -> None:
        _check(self._lib.avsg_set_transfer_geometry(self._h, blocks, threads), "avsg_set_transfer_geometry")

    def sync_status(self) -> int:
        """Waits for the device and returns the kernels' status word (0 = no problem was flagged)."""
        w = ctypes.c_uint32(0)
        rc = self._lib.avsg_sync_status(self._h, ctypes.byref(w))
        if rc != EDEVICE_STATUS:
            _check(rc, "avsg_sync_status")
        return w.value

    def clear_status(self) -> None:
        _check(self._lib.avsg_clear_status(self._h), "avsg_clear_status")

    def probe_wait_limit(self, stream=None) -> None:
        """Launches the overlapped transfer kernel alone (its Stage One never comes): it must give up by itself."""
        _check(self._lib.avsg_probe_wait_limit(self._h, _stream_handle(stream)), "avsg_probe_wait_limit")

    def stats(self) -> dict:
        s = AvsgStats()
        _check(self._lib.avsg_stats(self._h, ctypes.byref(s)), "avsg_stats")
        return {name: getattr(s, name) for name, _ in AvsgStats._fields_}

    def table_stats(self, table_id: int) -> dict:
        """Counters of one table (request-level hit rates are averaged from these)."""
        s = AvsgStats()
        _check(self._lib.avsg_table_stats(self._h, table_id, ctypes.byref(s)), "avsg_table_stats")
        return {name: getattr(s, name) for name, _ in AvsgStats._fields_ if not name.startswith("last_")}


def step_noalloc(tok, life, buffer, indices, kv, verified_len, *, max_lifetime: int = 16, slots, hit=None,
                 miss_count=None, status=None, row_stride=None, stream=None, kv_rows=None) -> None:
    """avsg_step_noalloc: one decode iteration on caller-owned state, for callers that cannot allocate
    (an engine whose own pool holds all device memory, or a path where an allocation's device-wide
    synchronisation is not acceptable).  Every tensor is the caller's; the library allocates nothing and
    keeps its scratch in a fixed array inside the library image.

    tok int32 [n, S], life int8 [n, S], buffer uint8 [n, S, row_bytes], indices int32 [n, n_tokens, topk],
    slots int32 like indices: CUDA tensors on the current device.  kv: one pinned host tensor (or address) per
    table.  Calls that overlap on the GPU race on the shared scratch: keep them on one stream.
    """
    n, S = tok.shape
    _, n_q, K = indices.shape
    kv_arr = (ctypes.c_void_p * n)(*[_addr(k) for k in kv])
    vlen = (ctypes.c_int32 * n)(*[int(v) for v in verified_len])
    stride = (ctypes.c_uint64 * n)(*[int(s) for s in row_stride]) if row_stride is not None else None
    a = AvsgNoAllocArgs()
    a.n, a.n_tokens, a.topk, a.buffer_slots = n, n_q, K, S
    a.row_bytes, a.max_lifetime = buffer.shape[-1], max_lifetime
    a.tok, a.life, a.buffer, a.indices = _addr(tok), _addr(life), _addr(buffer), _addr(indices)
    a.kv_base = ctypes.addressof(kv_arr)
    a.row_stride = ctypes.addressof(stride) if stride is not None else None
    a.verified_len = ctypes.addressof(vlen)
    a.slots = _addr(slots)
    a.hit = _addr(hit) if hit is not None else None
    a.miss_count = _addr(miss_count) if miss_count is not None else None
    a.status = _addr(status) if status is not None else None
    rows = (ctypes.c_uint32 * n)(*[int(r) for r in kv_rows]) if kv_rows is not None else None
    a.kv_rows = ctypes.addressof(rows) if rows is not None else None
    _check(load_library().avsg_step_noalloc(ctypes.byref(a), _stream_handle(stream)), "avsg_step_noalloc")
