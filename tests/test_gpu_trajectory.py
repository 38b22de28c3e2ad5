"""Lock-step trajectories: the CUDA path and the oracle run the whole schedule (prefill, decode,
eviction every E steps) on the same seeded stream.

Per step: out and the step's mass must agree within tolerance.  At each eviction the decision is
taken, on both sides, from the device's fp32 scores, and the device's compacted state must equal
the oracle's selection applied to the device's pre-eviction state bit for bit; the oracle's own
float64 scores are compared with the device's (<= 1e-4) just before, then re-synchronised so
that fp32 rounding drift does not accumulate across the whole run.
"""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def run_trajectory(cfg, seed, steps, cluster=0, variant=0, check_every=1):
    gpu = H.make_gpu(cfg, cluster, variant)
    orc = H.make_oracle(cfg)
    pk, pv = W.prompt_kv(cfg, seed)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64))
    stream = W.DecodeStream(cfg, seed)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=H.tdtype(cfg), device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    stats = dict(out=0.0, delta=0.0, score=0.0, events=0, moved=0)
    lengths = []
    for s in range(1, steps + 1):
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta)
        o_ref, d_ref = O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
        if s % check_every == 0 or s % cfg.evict_interval == 0:
            gpu.synchronize()
            stats["out"] = max(stats["out"], H.rel_err_vectors(out.float().cpu().numpy(), o_ref))
            dh = delta.cpu().numpy()
            for l, b, h, sl in orc.units():
                stats["delta"] = max(stats["delta"], float(np.abs(dh[l, b, h, :sl.n] - d_ref[l][b][h]).max()))
        if s % cfg.evict_interval == 0:
            sc = gpu.scores_tensor().cpu().numpy()
            for l, b, h, sl in orc.units():
                fin = np.isfinite(sl.score[:sl.n])
                stats["score"] = max(stats["score"], float(np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max()))
            n_before = gpu.len(0)
            kept = H.check_evict_bit_exact(gpu, cfg, cfg.budget)
            O.evict(orc, cfg.budget, scores32=lambda l, b, h: sc[l, b, h])
            sc2 = gpu.scores_tensor().cpu().numpy()
            for l, b, h, sl in orc.units():
                assert sl.n == gpu.len(b)
                sl.score[:sl.n] = sc2[l, b, h, :sl.n].astype(np.float64)     # re-synchronise
            if n_before > cfg.budget:
                stats["events"] += 1
                stats["moved"] += sum(int((np.asarray(kk) != np.arange(len(kk))).sum()) for kk in kept.values())
        lengths.append(gpu.len(0))
        assert gpu.len(0) == orc.length(0)
    gpu.poll_error()
    gpu.close()
    return stats, lengths


def test_config1_full_trajectory():
    """Config 1 exactly as stated: fp32, 4/1 heads, d 64, prompt 32, 512 steps, B 128, W 16, E 32."""
    cfg = W.get_config("c1_tiny_fp32")
    stats, lengths = run_trajectory(cfg, seed=1000, steps=cfg.decode_steps)
    assert stats["events"] == 13
    for i, n in enumerate(lengths, start=1):
        assert n == O.effective_length(cfg.prompt, i, cfg.budget + cfg.evict_interval, cfg.evict_interval)
    assert stats["out"] <= H.TOL_OUT["fp32"], stats
    assert stats["delta"] <= H.TOL_DELTA and stats["score"] <= H.TOL_DELTA, stats
    assert stats["moved"] > 0


@pytest.mark.parametrize("cluster", [1, 2, 4])
def test_config1_cluster_sizes(cluster):
    cfg = W.get_config("c1_tiny_fp32")
    stats, _ = run_trajectory(cfg, seed=1001, steps=200, cluster=cluster, variant=1)
    assert stats["out"] <= H.TOL_OUT["fp32"] and stats["delta"] <= H.TOL_DELTA and stats["score"] <= H.TOL_DELTA, stats


def test_config2_shortened():
    """Llama-8B head shapes and planted keys; layers, lengths and budget shortened."""
    cfg = W.get_config("c2_llama8b").scaled(layers=2, prompt=64, budget=384, window=32, evict_interval=32)
    stats, _ = run_trajectory(cfg, seed=2000, steps=480, check_every=7)
    assert stats["events"] == 480 // 32 - (384 - 64) // 32 + 0 or stats["events"] > 0
    assert stats["out"] <= H.TOL_OUT["bf16"] and stats["delta"] <= H.TOL_DELTA and stats["score"] <= H.TOL_DELTA, stats


def test_config3_shortened():
    """Qwen-7B head shapes (G = 7), batch 3."""
    cfg = W.get_config("c3_qwen7b").scaled(layers=2, batch=3, prompt=128, budget=512, window=64, evict_interval=64)
    stats, _ = run_trajectory(cfg, seed=3000, steps=640, check_every=13)
    assert stats["events"] > 0
    assert stats["out"] <= H.TOL_OUT["bf16"] and stats["delta"] <= H.TOL_DELTA and stats["score"] <= H.TOL_DELTA, stats


def test_config4_shortened_ragged():
    """Ragged batch: per-sequence budgets, sequences that finish early, heavy-tailed keys."""
    base = W.get_config("c4_ragged")
    cfg = base.scaled(layers=2, batch=4, prompt=32, window=16, evict_interval=32, seq_budgets=(96, 160, 224, 128),
                      budget=224, seq_decode_steps=(150, 400, 260, 90))
    gpu = H.make_gpu(cfg)
    orc = H.make_oracle(cfg)
    pk, pv = W.prompt_kv(cfg, 4000)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64))
    stream = W.DecodeStream(cfg, 4000)
    out = torch.zeros((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    active = [True] * cfg.batch
    worst = dict(out=0.0, delta=0.0)
    for s in range(1, max(cfg.seq_decode_steps) + 1):
        for b in range(cfg.batch):
            if active[b] and s > cfg.seq_decode_steps[b]:
                active[b] = False
                gpu.seq_reset(b)
                for l in range(cfg.layers):
                    for h in range(cfg.kv_heads):
                        orc.slab(l, b, h).n = 0
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta)
        o_ref, d_ref = O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), active=active)
        if s % 9 == 0 or s % cfg.evict_interval == 0:
            gpu.synchronize()
            og = out.float().cpu().numpy()
            dh = delta.cpu().numpy()
            for b in range(cfg.batch):
                if not active[b]:
                    continue
                worst["out"] = max(worst["out"], H.rel_err_vectors(og[:, b], o_ref[:, b]))
                for l in range(cfg.layers):
                    for h in range(cfg.kv_heads):
                        n = orc.slab(l, b, h).n
                        worst["delta"] = max(worst["delta"], float(np.abs(dh[l, b, h, :n] - d_ref[l][b][h]).max()))
        if s % cfg.evict_interval == 0:
            sc = gpu.scores_tensor().cpu().numpy()
            act = [(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch) if active[b] for h in range(cfg.kv_heads)]
            H.check_evict_bit_exact(gpu, cfg, 0, slabs=act)
            O.evict(orc, list(cfg.seq_budgets), scores32=lambda l, b, h: sc[l, b, h])
            sc2 = gpu.scores_tensor().cpu().numpy()
            for (l, b, h) in act:
                sl = orc.slab(l, b, h)
                sl.score[:sl.n] = sc2[l, b, h, :sl.n].astype(np.float64)
        for b in range(cfg.batch):
            assert gpu.len(b) == orc.slab(0, b, 0).n
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    gpu.poll_error()
    gpu.close()
