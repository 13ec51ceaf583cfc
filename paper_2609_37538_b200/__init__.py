"""AVSG per-decode-step operator for B200 (sm_100a): C-ABI library + thin Python binding."""
from .binding import (  # noqa: F401
    ECAPACITY, ECUDA, EDEVICE_STATUS, EINVAL, ENOMEM, EUNSUPPORTED, EXPORTS, OK, INDEX_DIRECT, INDEX_HASH, INDEX_PAPER,
    XFER_ALL_K, XFER_COPY_ENGINE, XFER_POSITION_LEVEL, XFER_REQUEST_LEVEL, XFER_SM_BALANCED, XFER_SM_OVERLAP,
    STATUS_BAD_ID, STATUS_BAD_SEGMENT, STATUS_BAD_SLOT, STATUS_NO_DEAD_SLOTS, STATUS_PROBE_EXHAUSTED, STATUS_WAIT_TIMEOUT,
    AvsgConfig, AvsgError, AvsgStats, AvsgStepArgs, Context, PreparedCall, StepOutput,
    load_library, pinned_empty, HostKV, HOST_KV_HUGE_PAGES,
    AvsgNoAllocArgs, NOALLOC_MAX_IDS, NOALLOC_MAX_TABLES, step_noalloc,
)
