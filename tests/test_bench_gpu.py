"""bench.py's own arm at a shrunk size on a GPU: the one JSON line carries every key of the contract."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("extra", [[], ["--stage-two", "balanced", "--index", "hash", "--host-kv", "huge"]])
def test_bench_line(extra):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--requests", "4", "--layers", "2", "--steps", "4", "--warmup", "3",
           "--replays", "20", "--tiny"] + extra
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
    assert r["peak_repeats"] == 4 and "numa_node" in d["numa"]
    assert d["one_call_per_step"]["tables_per_call"] == 8 and d["one_call_per_step"]["gbs"] > 0
    t = d["target"]
    assert 8 * 2048 <= t["cold_step"]["rows"] <= 8 * 4096 and 0 < t["cold_step"]["frac"] < 1.2   # token 0 misses everything
    assert set(t["met"]) == {"cold_step", "steady_call_stage_two_events", "steady_call_stage_two_in_kernel"}
    c5 = d["comparators_c5"]
    for mode in ("balanced", "request_level", "transfer_all_k"):
        assert c5[mode]["effective_gbs"] > 0 and c5[mode]["stage_two_us_per_iter"] > 0
    assert c5["transfer_all_k"]["raw_gbs"] > c5["transfer_all_k"]["effective_gbs"]      # it moves rows nobody needs


def _json_lines(args, timeout=900):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py")] + args
    out = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=timeout, check=True).stdout
    return [json.loads(l) for l in out.splitlines() if l.startswith("{")]


def test_suite_report_tiny():
    """bench.py --suite on shrunk shapes: every configuration reports, and so do the comparators."""
    rows = _json_lines(["--suite", "--tiny"])
    assert rows[0]["suite"] == "link" and rows[0]["link_peak_gbs"] > 1
    by = {(r["suite"], r.get("transfer_mode")): r for r in rows if "transfer_mode" in r}
    for name in ("C1", "C2", "C3", "C4", "C5"):
        r = by[(name, "sm_balanced")]
        assert 0 <= r["hit_rate"] <= 1 and r["cold_iter"]["rows"] > 0 and r["steady"]["transfer_us_per_iter"] > 0
    assert by[("C5", "request_level")]["steady"]["rows_per_iter"] == by[("C5", "sm_balanced")]["steady"]["rows_per_iter"]
    assert by[("C5", "transfer_all_k")]["steady"]["rows_per_iter"] > by[("C5", "sm_balanced")]["steady"]["rows_per_iter"]
    assert ("C3", "copy_engine") in by
    huge = by[("C4", "sm_balanced, host KV from avsg_host_kv_alloc")]
    assert huge["steady"]["rows_per_iter"] == by[("C4", "sm_balanced")]["steady"]["rows_per_iter"]
    assert 0 <= huge["host_kv_pages"]["huge_fraction"] <= 1
    modes = [r for r in rows if r["suite"] == "stage_two_modes"]
    assert len(modes) == 5 and all(set(m["us_per_iteration"]) == {"direct/balanced", "direct/overlap", "hash/balanced",
                                                                   "hash/overlap"} for m in modes)


def test_table3_report_tiny():
    """bench.py --table3 on a shrunk grid: with ONE request the miss-level split (S3) cannot be slower than one
    block serving the request alone (S1), which is the point of Eq. 6."""
    rows = _json_lines(["--table3", "--tiny", "--replays-table3", "1"])
    assert {(r["B"], r["reuse_pct"]) for r in rows} == {(1, 0), (1, 50), (4, 0), (4, 50)}
    for r in rows:
        assert r["rows"] == r["B"] * 256 * (100 - r["reuse_pct"]) // 100
        for k in ("S1_request_level_gbs", "S2_position_level_gbs", "S3_miss_level_gbs"):
            assert r[k] > 0
    one = [r for r in rows if r["B"] == 1 and r["reuse_pct"] == 0][0]
    assert one["S3_miss_level_gbs"] >= one["S1_request_level_gbs"]


def test_sweeps_report_tiny():
    rows = _json_lines(["--sweeps", "--tiny"])
    kinds = {r["sweep"] for r in rows}
    assert kinds == {"stage_one_latency", "lifetime", "capacity", "index_mode", "overlap_vs_tokens", "mtp_cold_start"}
    big = [r for r in rows if r["sweep"] == "stage_one_latency" and r["S"] == 16384]
    assert big and all(r["match_reserve_us_median"] > 0 for r in big)          # a pool only a cluster holds
    cold = {r["n_mtp"]: r["reuse"] for r in rows if r["sweep"] == "mtp_cold_start"}
    assert cold[0] == 0 and cold[3] > 0                                          # later tokens reuse earlier ones' rows
    idx = {r["index"]: r["hit_rate"] for r in rows if r["sweep"] == "index_mode"}
    assert idx["exact_hash"] == idx["exact_direct"] >= idx["paper_R3"]


def test_breakdown_report_tiny():
    rows = [r for r in _json_lines(["--breakdown", "--tiny"]) if r["breakdown"] != "link"]
    assert len(rows) == 8 and {r["stage_two"] for r in rows} == {"overlap", "balanced"}
    for r in rows:
        sp = r["split_us"]
        assert r["rows_per_call"] > 0 and r["event_us_per_call"] > 0
        assert sp["stage_one_exposed"] > 0 and sp["first_row"] >= 0 and sp["copy"] >= 0 and sp["tail"] >= 0
        assert abs(sum(sp.values()) - r["event_us_per_call"]) < 0.05 * r["event_us_per_call"] + 1.0


def test_link_model_report_tiny():
    rows = _json_lines(["--link-model", "--tiny"])
    fit = [r for r in rows if r["link_model"] == "fit"][0]
    assert fit["link_peak_gbs"] > 1 and "raw_rate_gbs_R" in fit and "header_bytes_H" in fit    # (no fit at this size)
    assert len([r for r in rows if r["link_model"] == "span"]) == 2
    geo = {(r["row_bytes"], r["row_stride"]): r for r in rows if r["link_model"] is True}
    assert set(geo) == {(656, 656), (656, 768), (1152, 1152)}
    assert geo[(1152, 1152)]["sectors_per_row"] == 36 and geo[(1152, 1152)]["lines_per_row"] == 9
    assert geo[(656, 768)]["sectors_per_row"] == 21 and geo[(656, 768)]["lines_per_row"] == 6
    assert geo[(656, 656)]["lines_per_row"] == 6 and 21 <= geo[(656, 656)]["sectors_per_row"] <= 22
