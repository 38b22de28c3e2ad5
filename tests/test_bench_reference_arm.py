"""CPU checks of bench.py's reference arm (the float64 oracle timed on the host cores): the JSON
contract of the line, and the N > 1 launch, where rank 0 alone works and prints and the other
ranks exit 0 without work.  The hot path itself does not shard (replicas only), so there is no
collective to test; this covers the launch logic with two CPU processes."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ARGS = ["bench.py", "--impl", "reference", "--workload", "c1_tiny_fp32", "--steps", "3", "--warmup", "1"]


def _check_line(line, n_gpus):
    d = json.loads(line)
    assert d["impl"] == "reference" and d["n_gpus"] == n_gpus and d["steps"] == 3 and d["warmup"] == 1
    assert d["metric"] == "decode tokens/s at budget B" and d["unit"] == "tokens/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["config"]["workload"] == "c1_tiny_fp32" and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    # the same description of the workload as the main arm prints (bench.workload_config)
    assert set(d["config"]) == {"workload", "layers", "batch", "q_heads", "kv_heads", "head_dim", "budget", "window",
                                "evict_interval", "prompt_pinned", "dist", "score_source", "selection", "kv_dtype",
                                "kv_bytes", "l2_policy", "replicas"}
    assert d["config"]["replicas"] == n_gpus


def test_reference_arm_single_process():
    res = subprocess.run([sys.executable] + ARGS, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    _check_line(lines[0], 1)


def test_reference_arm_two_ranks_only_rank0_prints():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29731"] + ARGS + ["--gpus", "2"]
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    res = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    _check_line(lines[0], 2)
