"""GPU parity of the eviction (Section 4.2): selection decisions and compacted K/V/pos/score must
equal the oracle's, bit for bit, when both decide from the same fp32 scores."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _filled(cfg, rows, n_pinned, seed):
    gpu = H.make_gpu(cfg)
    k, v = W.prompt_kv(cfg, seed, n_tokens=rows)
    gpu.prefill(H.dev(k, cfg), H.dev(v, cfg), n_pinned=n_pinned)
    return gpu


def _set_scores(gpu, cfg, rows, n_pinned, fn, seed=0):
    """Overwrite the device scores of the unpinned rows (the external-score path)."""
    sc = gpu.scores_tensor()
    rng = np.random.default_rng(seed)
    vals = fn(rng, (cfg.layers, cfg.batch, cfg.kv_heads, rows - n_pinned)).astype(np.float32)
    sc[..., n_pinned:rows] = torch.from_numpy(vals).to(sc.device)
    torch.cuda.synchronize()


PATTERNS = {
    "random": lambda r, s: r.random(s),
    "all_equal": lambda r, s: np.zeros(s),
    "few_levels_many_ties": lambda r, s: r.integers(0, 4, s) / 4.0,
    "ascending": lambda r, s: np.broadcast_to(np.arange(s[-1], dtype=np.float64), s).copy(),
    "descending": lambda r, s: np.broadcast_to(np.arange(s[-1], 0, -1, dtype=np.float64), s).copy(),
    "negative_and_zero": lambda r, s: np.where(r.random(s) < 0.3, -0.0, r.standard_normal(s)),
    "tiny_denormal_mix": lambda r, s: r.random(s) * 1e-40,
    "huge_and_inf": lambda r, s: np.where(r.random(s) < 0.05, np.inf, r.random(s) * 1e30),
    "first_candidate_lowest": lambda r, s: np.concatenate([np.full(s[:-1] + (1,), -1.0), 1 + r.random(s[:-1] + (s[-1] - 1,))], -1),
    "every_other": lambda r, s: np.broadcast_to((np.arange(s[-1]) % 2).astype(np.float64), s).copy(),
    "block_before_window_lowest": lambda r, s: np.concatenate([1 + r.random(s[:-1] + (s[-1] - 40,)), np.zeros(s[:-1] + (40,))], -1),
}


@pytest.mark.parametrize("pattern", sorted(PATTERNS))
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("fp32", 64), ("fp32", 96), ("bf16", 256), ("fp32", 256)])
def test_patterns_bit_exact(pattern, dtype, d):
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=2, kv_heads=2, q_heads=8, head_dim=d, dtype=dtype,
                                             prompt=24, budget=700, window=32, evict_interval=600)
    rows = 1237                                     # several 1024-thread chunks and a ragged tail
    gpu = _filled(cfg, rows, cfg.prompt, seed=1)
    _set_scores(gpu, cfg, rows, cfg.prompt, PATTERNS[pattern], seed=2)
    kept = H.check_evict_bit_exact(gpu, cfg, cfg.budget)
    assert all(len(k) == cfg.budget for k in kept.values())
    assert gpu.len(0) == cfg.budget
    # idempotent
    again = H.check_evict_bit_exact(gpu, cfg, cfg.budget)
    assert all(list(k) == list(range(cfg.budget)) for k in again.values())
    gpu.close()


@pytest.mark.parametrize("split", [-1, 1, 2, 4, 8])
@pytest.mark.parametrize("pattern", ["random", "all_equal", "few_levels_many_ties", "negative_and_zero", "first_candidate_lowest",
                                     "block_before_window_lowest"])
@pytest.mark.parametrize("dtype,d,rows,budget", [("bf16", 128, 1237, 700), ("fp32", 96, 1000, 300), ("bf16", 128, 2112, 2048),
                                                 ("bf16", 128, 3136, 3072), ("bf16", 128, 4224, 4096), ("bf16", 128, 4352, 1000)])
def test_ctas_per_slab_and_row_count_tiers(split, pattern, dtype, d, rows, budget):
    """The eviction kernel's launch shapes: one CTA per slab with shared-memory keys (-1), or 1, 2,
    4, 8 CTAs per slab that each decide for themselves and move a share of the row bytes; row
    counts in each of the kernel's register tiers (up to 1280, 2304, 3328, 4352 rows)."""
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=2, kv_heads=2, q_heads=8, head_dim=d, dtype=dtype,
                                             prompt=24, budget=budget, window=32, evict_interval=rows - budget)
    gpu = _filled(cfg, rows, cfg.prompt, seed=1)
    gpu.set_evict_launch(split)
    _set_scores(gpu, cfg, rows, cfg.prompt, PATTERNS[pattern], seed=2)
    kept = H.check_evict_bit_exact(gpu, cfg, cfg.budget)
    assert all(len(k) == cfg.budget for k in kept.values()) and gpu.len(1) == cfg.budget
    rows_scanned, rows_moved = gpu.evict_stats()
    assert rows_scanned == rows * 8
    assert rows_moved == sum(cfg.budget - int(np.flatnonzero(k != np.arange(len(k)))[0]) if (k != np.arange(len(k))).any() else 0
                             for k in kept.values())
    gpu.close()


@pytest.mark.parametrize("target", [56, 57, 100, 699, 1236, 1237, 5000])
def test_targets_from_window_only_to_no_op(target):
    """k = 0 (question + local window only) ... target >= n (nothing moves)."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=24, budget=700, window=32, evict_interval=600)
    gpu = _filled(cfg, 1237, 24, seed=3)
    _set_scores(gpu, cfg, 1237, 24, PATTERNS["random"], seed=target)
    kept = H.check_evict_bit_exact(gpu, cfg, target)
    assert gpu.len(0) == min(1237, target)
    if target == 56:
        assert list(kept[(0, 0, 0)]) == list(range(24)) + list(range(1237 - 32, 1237))
    gpu.close()


def test_budget_error_leaves_cache_unchanged():
    import paper_2601_18383_b200 as D
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=24, budget=700, window=32, evict_interval=600)
    gpu = _filled(cfg, 300, 24, seed=4)
    with pytest.raises(D.DyntsError) as e:
        gpu.evict(55)
    assert e.value.status == D.DYNTS_ERR_BUDGET and gpu.len(0) == 300
    gpu.close()


def test_no_pins_no_window_pure_topk():
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=0, budget=64, window=0, evict_interval=600)
    gpu = _filled(cfg, 500, 0, seed=5)
    _set_scores(gpu, cfg, 500, 0, PATTERNS["random"], seed=5)
    s0 = gpu.export_slab(0, 0, 0)[3].numpy()
    kept = H.check_evict_bit_exact(gpu, cfg, 64, pinned=[0])
    assert set(kept[(0, 0, 0)]) == set(np.argsort(-s0, kind="stable")[:64])
    gpu.close()


def test_per_sequence_targets_and_lengths():
    cfg = W.get_config("c4_ragged").scaled(layers=2, batch=4, prompt=16, window=8, evict_interval=64,
                                            seq_budgets=(100, 300, 200, 1000), seq_decode_steps=None, budget=1000)
    gpu = H.make_gpu(cfg)
    rows = [250, 310, 150, 400]
    for b, r in enumerate(rows):
        k, v = W.prompt_kv(cfg.scaled(batch=1), 10 + b, n_tokens=r)
        gpu.prefill_seq(b, H.dev(k[:, 0], cfg), H.dev(v[:, 0], cfg), n_pinned=16)
    sc = gpu.scores_tensor()
    sc[..., 16:] = torch.rand(sc[..., 16:].shape, device=sc.device)
    torch.cuda.synchronize()
    assert [gpu.len(b) for b in range(4)] == rows
    H.check_evict_bit_exact(gpu, cfg, 0, pinned=[16] * 4)        # configured per-sequence budgets
    assert [gpu.len(b) for b in range(4)] == [100, 300, 150, 400]
    H.check_evict_bit_exact(gpu, cfg, [50, 50, 50, 50], pinned=[16] * 4)
    assert [gpu.len(b) for b in range(4)] == [50, 50, 50, 50]
    gpu.close()


def test_attention_after_eviction_matches_oracle_on_compacted_state():
    """The compacted cache is a valid cache: the next decode step matches the oracle run from the
    exported post-eviction state."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=32, budget=256, window=16, evict_interval=64)
    gpu = _filled(cfg, 300, 32, seed=6)
    _set_scores(gpu, cfg, 300, 32, PATTERNS["random"], seed=6)
    gpu.evict(0)
    orc = H.oracle_from_gpu(gpu, cfg)
    q, k, v = W.DecodeStream(cfg, 6).step(1)
    out = torch.empty((1, 1, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out)
    o_ref, _ = O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
    assert H.rel_err_vectors(out.float().cpu().numpy(), o_ref) <= H.TOL_OUT["bf16"]
    pos = gpu.export_slab(0, 0, 0)[2].numpy()
    assert pos[-1] == 300 and (np.diff(pos) > 0).all()
    gpu.close()
