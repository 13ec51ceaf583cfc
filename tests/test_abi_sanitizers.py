"""The C ABI's argument paths under AddressSanitizer and UndefinedBehaviorSanitizer, on the host, without a GPU.

A second build of the library has its HOST code instrumented (nvcc hands -fsanitize to the host compiler; device
code is unchanged) and a small C program (tests/abi/abi_driver.c, instrumented too) walks the entry points with
arguments that must be refused.  The same program prints the layout of the public structs as the C compiler sees
them, which is compared with the binding's ctypes structures."""
import ctypes
import glob
import os
import subprocess

import pytest

import paper_2609_37538_b200 as avsg
from paper_2609_37538_b200 import build as pkg_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAN = ["-fsanitize=address", "-fsanitize=undefined", "-fno-omit-frame-pointer", "-fno-sanitize-recover=undefined"]


@pytest.fixture(scope="module")
def driver_output(tmp_path_factory):
    tmp = tmp_path_factory.mktemp("abi_san")
    lib, exe = tmp / "libavsg_san.so", tmp / "abi_driver"
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [f for f in pkg_build.NVCC_FLAGS if f != "-O3"] + ["-O1", "-g"]
    host = [x for f in SAN for x in ("-Xcompiler", f)]      # one by one: nvcc splits -Xcompiler values at commas
    subprocess.check_call([nvcc] + flags + host + ["-I", pkg_build.INCLUDE, "-I", pkg_build.CSRC, "-o", str(lib)]
                          + [s for s in pkg_build.sources() if s.endswith(("avsg_api.cu", "no_alloc.cu"))]
                          + [s for s in pkg_build.sources() if not s.endswith(("avsg_api.cu", "no_alloc.cu"))])
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-g"] + SAN + ["-I", pkg_build.INCLUDE,
                                                                                  os.path.join(ROOT, "tests", "abi", "abi_driver.c"),
                                                                                  "-o", str(exe), str(lib), "-Wl,-rpath," + str(tmp)])
    env = dict(os.environ, ASAN_OPTIONS="detect_leaks=0:abort_on_error=0:protect_shadow_gap=0",
               UBSAN_OPTIONS="print_stacktrace=1:halt_on_error=1", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([str(exe)], env=env, capture_output=True, text=True, timeout=300)
    return r


def test_argument_paths_are_clean_under_asan_and_ubsan(driver_output):
    r = driver_output
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    assert "failures 0" in r.stdout
    assert "ERROR: AddressSanitizer" not in r.stderr and "runtime error:" not in r.stderr, r.stderr[-3000:]


def test_ctypes_layouts_equal_the_c_compilers(driver_output):
    facts = {}
    for line in driver_output.stdout.splitlines():
        kind, name, value = (line.split() + [None, None])[:3]
        if kind in ("sizeof", "offsetof"):
            facts[(kind, name)] = int(value)
    assert facts[("sizeof", "avsg_config")] == ctypes.sizeof(avsg.AvsgConfig)
    assert facts[("sizeof", "avsg_step_args")] == ctypes.sizeof(avsg.AvsgStepArgs)
    assert facts[("sizeof", "avsg_stats_t")] == ctypes.sizeof(avsg.AvsgStats)
    assert facts[("sizeof", "avsg_noalloc_args")] == ctypes.sizeof(avsg.AvsgNoAllocArgs)
    assert facts[("offsetof", "avsg_config.stage_one_cluster")] == avsg.AvsgConfig.stage_one_cluster.offset
    assert facts[("offsetof", "avsg_step_args.kv_rows")] == avsg.AvsgStepArgs.kv_rows.offset
    assert facts[("offsetof", "avsg_step_args.indices")] == avsg.AvsgStepArgs.indices.offset
    assert facts[("offsetof", "avsg_noalloc_args.kv_rows")] == avsg.AvsgNoAllocArgs.kv_rows.offset
    assert facts[("offsetof", "avsg_stats_t.last_rows")] == avsg.AvsgStats.last_rows.offset
