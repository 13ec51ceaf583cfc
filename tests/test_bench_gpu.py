"""bench.py's own arm at a shrunk size on a GPU: the one JSON line carries every key of the contract."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("extra", [[], ["--stage-two", "balanced", "--index", "hash"]])
def test_bench_line(extra):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--requests", "4", "--layers", "2", "--steps", "4", "--warmup", "3",
           "--replays", "20"] + extra
    out = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=900, check=True).stdout
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] == 3 and d["value"] > 0
    assert d["gpu_launches"] == 2 * 2 * 4                       # two kernels per call, two calls per step, four steps
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    r = d["roofline"]
    assert r["bound"] == "host_link" and r["unit"] == "GB/s" and 0 < r["frac"] == pytest.approx(r["achieved"] / r["peak"])
    assert r["traffic"] > 0 and r["kernel"].startswith("avsg_transfer")
    assert d["roofline_stage_one"]["bound"] == "hbm" and d["roofline_stage_one"]["peak"] > 1000
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] > 0
    assert d["clocks"]["sm_max_mhz"] >= d["clocks"]["sm_mhz"] > 0
    assert 0.5 < d["hit_rate"] < 1.0 and d["config"]["workload"].startswith("C3")
