"""The N > 1 launch of the benchmark on two CPU processes (gloo): the hot path shards by giving every
rank its own batch of sequences and exchanges nothing, so what there is to test is the host logic
around it -- distinct data per rank, the slowest rank's time as the job's time, the whole-job
throughput, one printed line."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = textwrap.dedent("""
    import json, os, sys
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.getcwd())
    import bench
    import workloads as W

    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    cfg = W.get_config("c1_tiny_fp32")
    seed = bench.rank_seed(cfg, rank)
    # this rank's shard of the job: its own prompt rows and its own decode stream
    k, v = W.prompt_kv(cfg, seed, n_tokens=cfg.prompt)
    q1, k1, v1 = W.DecodeStream(cfg, seed).step(1)
    digest = float(np.abs(k).sum() + np.abs(q1).sum())
    # every rank measured its own time; the job took as long as the slowest
    my_ms = 10.0 * (rank + 1)
    job_ms = bench.max_over_ranks(my_ms, world)
    # digests of all ranks, to show that the shards differ
    box = [None] * world
    dist.all_gather_object(box, (seed, digest))
    value = bench.job_throughput(cfg.batch, 7, world, job_ms * 1e-3)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"job_ms": job_ms, "value": value, "shards": box, "n_gpus": world}), flush=True)
    dist.destroy_process_group()
""")


def test_two_ranks_shard_the_batch_and_report_the_slowest_rank(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(RANK_SCRIPT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29741", str(script)]
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    res = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout          # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2
    assert d["job_ms"] == 20.0                  # the maximum over the ranks, not rank 0's own 10 ms
    assert abs(d["value"] - 1 * 7 * 2 / 20e-3) < 1e-9    # batch x steps x ranks / the job's time
    (s0, g0), (s1, g1) = d["shards"]
    assert s0 != s1 and g0 != g1                # different seeds, different rows: the ranks hold different sequences


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.job_throughput(16, 128, 1, 0.5) == 16 * 128 / 0.5
