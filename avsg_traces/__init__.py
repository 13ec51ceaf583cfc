"""Seeded synthetic inputs shared by the oracle's tests and the CUDA path's tests.

Holds the trace generator (DSA-shaped top-K selections) and the host KV byte
generator.  Nothing here performs any step of the operator itself.
"""
from .gen import (  # noqa: F401
    TraceConfig,
    Workload,
    build_library,
    fill_kv,
    generate,
    kv_rows,
    workload,
    WORKLOADS,
)
