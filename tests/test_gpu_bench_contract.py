"""The benchmark's JSON line on a GPU: the keys and invariants its consumers rely on (a short run
on the tiny workload and on a shortened default workload)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra, steps=128, warmup=64):
    cmd = [sys.executable, "bench.py", "--steps", str(steps), "--warmup", str(warmup), "--cpu-seconds", "1",
           "--sustain-seconds", "0.3"] + list(extra)
    res = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


@pytest.mark.parametrize("extra", [(), ("--score-source", "external"), ("--workload", "c1_tiny_fp32")])
def test_bench_line_contract(extra):
    d = _run(*extra)
    assert d["metric"] == "decode tokens/s at budget B" and d["unit"] == "tokens/s" and d["higher_is_better"] is True
    assert d["n_gpus"] == 1 and d["steps"] == 128 and d["warmup"] == 64 and d["run"]["warmup_steps_run"] >= 64 and d["scaling"] == "weak"
    assert d["vs_baseline"] is None and d["data"] == "synthetic" and d["dtype"] in ("bf16", "f32")
    assert d["value"] > 0 and abs(d["value"] - d["config"]["batch"] / (d["ms_per_step"] * 1e-3)) <= 0.01 * d["value"]
    assert "workload" in d["config"] and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and r["achieved"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3 and "traffic" in r
    e = d["e2e"]
    assert e["value"] > 0 and e["unit"] == "tokens/s" and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"] * 1.05                      # the end-to-end arm includes the copies
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    assert d["gpu_launches"] >= 128
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    _check_cycle_keys(d)


def _check_cycle_keys(d):
    """The eviction half of the metric is in the line whatever the step count: at least four timed
    events, a whole cycle (E decode steps + 1 eviction), a sustained region with its clocks, and an
    end-to-end arm that contains an eviction."""
    E = d["config"]["evict_interval"]
    ev = d["evict"]
    assert ev["bound"] == "hbm" and ev["events_timed"] >= 4 and ev["avg_event_us"] > 0 and ev["algorithmic_bytes_per_event"] > 0
    assert abs(ev["frac"] - ev["achieved"] / ev["peak"]) < 1e-3
    assert abs(ev["evict_per_step_us"] - ev["avg_event_us"] / E) < 1e-2
    cy = d["cycle"]
    assert cy["decode_steps"] == E and cy["evictions"] == 1 and cy["tokens_per_s"] > 0 and cy["cycles_timed"] >= 4
    assert abs(cy["tokens_per_s"] - d["config"]["batch"] * E / (cy["ms"] * 1e-3)) <= 0.01 * cy["tokens_per_s"]
    su = d["sustained"]
    assert su["seconds"] >= 0.25 and su["steps"] == su["cycles"] * E and su["tokens_per_s"] > 0
    assert set(su["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert sum(b["cycles"] for b in su["by_sm_mhz"]) in (0, su["cycles"])
    e = d["e2e"]
    assert e["steps"] % E == 0 and e["evictions"] == e["steps"] // E >= 1
    assert d["run"]["evictions_in_timed_region"] == d["steps"] // E


@pytest.mark.parametrize("steps,warmup", [(100, 5), (2, 1), (70, 3)])
def test_step_counts_off_the_eviction_cycle(steps, warmup):
    """K and W need not be multiples of the eviction interval: the eviction cycle carries over from
    the timed region into the per-kernel pass and the end-to-end arm."""
    d = _run("--no-cpu-baseline", steps=steps, warmup=warmup)
    assert d["steps"] == steps and d["warmup"] == warmup and d["run"]["warmup_steps_run"] >= max(3, warmup)
    assert d["value"] > 0 and d["roofline"]["achieved"] > 0 and d["e2e"]["value"] > 0
    assert d["gpu_launches"] >= steps
    _check_cycle_keys(d)


def test_both_arms_describe_the_workload_alike():
    ours = _run("--no-cpu-baseline", "--no-extras", steps=20, warmup=5)
    cmd = [sys.executable, "bench.py", "--impl", "reference", "--steps", "2", "--warmup", "1"]
    res = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-3000:]
    ref = json.loads([l for l in res.stdout.splitlines() if l.startswith("{")][0])
    assert ref["config"] == ours["config"] and ref["metric"] == ours["metric"] and ref["unit"] == ours["unit"]
