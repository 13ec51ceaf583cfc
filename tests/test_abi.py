"""The C-ABI library loads without a GPU and exports every symbol include/avsg.h declares."""
import ctypes
import os
import re

import paper_2609_37538_b200 as avsg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "avsg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(avsg_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree():
    assert _declared() == sorted(avsg.EXPORTS)


def test_library_exports_every_declared_symbol():
    lib = avsg.load_library()
    for name in _declared():
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(avsg.AvsgConfig) == 56
    assert ctypes.sizeof(avsg.AvsgStepArgs) == 120
    assert ctypes.sizeof(avsg.AvsgStats) == 104
    assert ctypes.sizeof(avsg.AvsgNoAllocArgs) == 120


def test_error_strings_and_argument_errors_need_no_gpu():
    lib = avsg.load_library()
    for code in (0, -1, -2, -3, -4, -5, -6):
        assert lib.avsg_strerror(code)
    assert lib.avsg_strerror(-99) == b"unknown error"
    h = ctypes.c_void_p()
    assert lib.avsg_create(None, ctypes.byref(h)) == avsg.EINVAL
    bad = avsg.AvsgConfig(1, 1000, 656, 16, 1, 16, 0, 0)            # slots not a power of two
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EINVAL
    bad = avsg.AvsgConfig(1, 1024, 650, 16, 1, 16, 0, 0)            # row bytes not a multiple of 16
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EINVAL
    bad = avsg.AvsgConfig(1, 1024, 656, 600, 2, 16, 0, 0)           # Eq. 7: 2 * 600 > 1024
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.ECAPACITY
    bad = avsg.AvsgConfig(1, 65536, 656, 2048, 2, 16, 0, 0)         # more slots than a cluster holds
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EUNSUPPORTED
    bad = avsg.AvsgConfig(1, 1024, 656, 16, 1, 16, 0, 0, 0, 0, 0, 0, 0, 3)       # cluster size not a power of two
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EINVAL
    bad = avsg.AvsgConfig(1, 1024, 656, 16, 1, 200, 0, 0)
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EINVAL
    assert lib.avsg_step(None, None, None) == avsg.EINVAL
    assert lib.avsg_destroy(None) == avsg.EINVAL
    bad = avsg.AvsgConfig(1, 1024, 656, 16, 1, 16, 6, 0)            # transfer mode beyond the last one
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EINVAL
    bad = avsg.AvsgConfig(1, 1024, 656, 16, 1, 16, 0, 0, avsg.INDEX_DIRECT, 0)   # direct index without max_context
    assert lib.avsg_create(ctypes.byref(bad), ctypes.byref(h)) == avsg.EINVAL
    st = avsg.AvsgStats()
    for call in (lambda: lib.avsg_stats(None, ctypes.byref(st)), lambda: lib.avsg_table_stats(None, 0, ctypes.byref(st)),
                 lambda: lib.avsg_sync_status(None, None), lambda: lib.avsg_clear_status(None),
                 lambda: lib.avsg_probe_wait_limit(None, None), lambda: lib.avsg_set_transfer_mode(None, 0),
                 lambda: lib.avsg_set_timing(None, 1), lambda: lib.avsg_set_transfer_geometry(None, 148, 256),
                 lambda: lib.avsg_save_state(None, None), lambda: lib.avsg_restore_state(None, None),
                 lambda: lib.avsg_reset(None, None, 0), lambda: lib.avsg_step_host(None, None, None)):
        assert call() == avsg.EINVAL
    p = ctypes.c_void_p()
    assert lib.avsg_host_kv_alloc(0, 0, ctypes.byref(p), None) == avsg.EINVAL          # no bytes
    assert lib.avsg_host_kv_alloc(4096, 2, ctypes.byref(p), None) == avsg.EINVAL       # unknown flag
    assert lib.avsg_host_kv_alloc(4096, 0, None, None) == avsg.EINVAL                  # nowhere to put the address
    assert lib.avsg_host_kv_alloc(1 << 60, 0, ctypes.byref(p), None) == avsg.EINVAL    # beyond any address space
    assert lib.avsg_host_kv_free(None) == avsg.EINVAL
    assert lib.avsg_host_kv_free(ctypes.c_void_p(4096)) == avsg.EINVAL                 # not from the allocator


def test_product_sources_do_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_37538_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower().replace("no cpu fallback", ""), f
