"""GPU parity of the paper's inference mode (Section 4.1-4.2): importance scores supplied per token
by a predictor (here: seeded random numbers standing in for its output), appended beside the KV,
selection triggered when the row count reaches the budget B and keeping a ratio of the selection
window.  The scores are exact float32 inputs on both sides, so the whole trajectory -- retained
positions, K, V, scores -- must equal the oracle's bit for bit; attention outputs within tolerance."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _scores(seed, s, batch):
    return np.random.default_rng([seed, s]).standard_normal(batch).astype(np.float32)


@pytest.mark.parametrize("name,variant,ratio", [("c2_llama8b", 0, 0.4), ("c2_llama8b", 2, 0.3), ("c3_qwen7b", 0, 0.4),
                                                 ("c1_tiny_fp32", 0, 0.5)])
def test_predictor_scores_and_trigger_at_budget(name, variant, ratio):
    import paper_2601_18383_b200 as D
    B = 160
    cfg = W.get_config(name).scaled(layers=2, batch=2, prompt=40, budget=B, window=24, evict_interval=1,
                                    **({"kv_heads": 2, "q_heads": 14} if name == "c3_qwen7b" else {}))
    gpu = H.make_gpu(cfg, 0, variant)
    gpu.set_score_source(D.DYNTS_SCORE_EXTERNAL)
    orc = H.make_oracle(cfg)
    pk, pv = W.prompt_kv(cfg, 21)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64))
    stream = W.DecodeStream(cfg, 21)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=H.tdtype(cfg), device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    M = cfg.prompt
    K_evicted = (B - M - cfg.window) - int(np.floor(ratio * (B - M - cfg.window)))
    worst_out = worst_delta = 0.0
    events = 0
    for s in range(1, 301):
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta)
        sn = _scores(77, s, cfg.batch)
        gpu.append_scores(torch.from_numpy(sn).cuda())
        o_ref, d_ref = O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), accumulate=False)
        O.set_new_scores(orc, sn)
        if s % 11 == 0:
            gpu.synchronize()
            worst_out = max(worst_out, H.rel_err_vectors(out.float().cpu().numpy(), o_ref))
            dh = delta.cpu().numpy()
            for l, b, h, sl in orc.units():
                worst_delta = max(worst_delta, float(np.abs(dh[l, b, h, :sl.n] - d_ref[l][b][h]).max()))
        n_before = gpu.len(0)
        gpu.evict_at_budget(B, ratio)
        if orc.length(0) >= B:
            O.evict(orc, O.paper_target(M, B, cfg.window, ratio))
            events += 1
        assert gpu.len(0) == orc.length(0) == O.effective_length(M, s, B, K_evicted), (s, n_before)
        if n_before >= B or s == 300:
            for l, b, h, sl in orc.units():
                Kd, Vd, pos, score = gpu.export_slab(l, b, h)
                assert np.array_equal(pos.numpy(), sl.pos[:sl.n])
                assert np.array_equal(score.numpy().astype(np.float64), sl.score[:sl.n])
                assert np.array_equal(Kd.to(torch.float64).numpy(), sl.K[:sl.n])
                assert np.array_equal(Vd.to(torch.float64).numpy(), sl.V[:sl.n])
    gpu.poll_error()
    assert events >= 3
    # one retained set per sequence (the scores are shared by all layers and heads)
    for b in range(cfg.batch):
        ref = gpu.export_slab(0, b, 0)[2]
        for l in range(cfg.layers):
            for h in range(cfg.kv_heads):
                assert torch.equal(gpu.export_slab(l, b, h)[2], ref)
    assert worst_out <= H.TOL_OUT[cfg.dtype] and worst_delta <= H.TOL_DELTA, (worst_out, worst_delta)
    gpu.close()


def test_external_mode_without_delta_output_and_argument_checks():
    import paper_2601_18383_b200 as D
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=30, budget=64, window=8, evict_interval=4)
    gpu = H.make_gpu(cfg)
    with pytest.raises(D.DyntsError):
        gpu.set_score_source(7)
    gpu.set_score_source(D.DYNTS_SCORE_EXTERNAL)
    pk, pv = W.prompt_kv(cfg, 3)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg), n_pinned=10)
    stream = W.DecodeStream(cfg, 3)
    out = torch.empty((1, 1, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    before = gpu.scores_tensor().clone()
    q, k, v = [H.dev(x, cfg) for x in stream.step(1)]
    gpu.decode_attn(q, k, v, out)                       # no delta buffer: the logit scratch is skipped
    gpu.synchronize()
    after = gpu.scores_tensor()
    assert torch.equal(after[..., :30].view(torch.int32), before[..., :30].view(torch.int32))
    assert (after[..., 30] == 0).all()
    gpu.append_scores(torch.tensor([1.5], device="cuda:0"))
    gpu.synchronize()
    assert (gpu.scores_tensor()[..., 30] == 1.5).all()
    with pytest.raises(D.DyntsError):
        gpu.evict_at_budget(10 ** 6, 0.5)               # beyond the capacity
    with pytest.raises(D.DyntsError):
        gpu.evict_at_budget(40, 1.5)
    gpu.evict_at_budget(40, 0.5)                        # 31 rows < 40: nothing happens
    assert gpu.len(0) == 31
    gpu.close()


@pytest.mark.parametrize("name", ["c2_llama8b", "c3_qwen7b", "c1_tiny_fp32"])
def test_sequence_wide_selection_on_aggregated_scores(name):
    """Attention mass accumulates per slab; at every eviction the slab scores of a sequence are
    summed (Appendix B.1) and one selection per sequence is applied to all layers and heads.  The
    oracle repeats the decision from the device's own float32 scores: the compacted state of every
    slab must then be bit-identical."""
    extra = {"kv_heads": 2, "q_heads": 14} if name == "c3_qwen7b" else {}
    cfg = W.get_config(name).scaled(layers=3, batch=2, prompt=24, budget=96, window=16, evict_interval=32, **extra)
    gpu, orc = H.make_gpu(cfg), H.make_oracle(cfg)
    pk, pv = W.prompt_kv(cfg, 31)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64))
    stream = W.DecodeStream(cfg, 31)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=H.tdtype(cfg), device="cuda:0")
    events = moved = 0
    worst_score = worst_key = 0.0
    for s in range(1, 225):
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out)
        O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
        if s % cfg.evict_interval:
            continue
        sc = gpu.scores_tensor().cpu().numpy()
        pre = H.export_all(gpu, cfg)
        for l, b, h, sl in orc.units():
            fin = np.isfinite(sl.score[:sl.n])
            worst_score = max(worst_score, float(np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max()))
        n_before = gpu.len(0)
        # the device's aggregated keys: within rounding of the float64 sum of its own slab scores
        # (Appendix B.1), and the array the oracle's selection is taken from
        keys_t = torch.full((cfg.batch, gpu.capacity), float("nan"), dtype=torch.float32, device="cuda:0")
        gpu.aggregate_scores(keys_t)
        keys = keys_t.cpu().numpy()
        n_slabs = cfg.layers * cfg.kv_heads
        for b in range(cfg.batch):
            exact = sc[:, b, :, :n_before].astype(np.float64).sum(axis=(0, 1))
            fin = np.isfinite(exact)
            assert np.array_equal(np.isinf(keys[b, :n_before]), ~fin)
            worst_key = max(worst_key, float(np.abs(keys[b, :n_before][fin] - exact[fin]).max()))
            assert np.isnan(keys[b, n_before:]).all()              # rows beyond the length are left alone
        gpu.evict_global(0)
        gpu.synchronize()
        gpu.poll_error()
        kept = O.evict_global(orc, cfg.budget, keys32=lambda b: keys[b])
        for l, b, h, sl in orc.units():
            K0, V0, p0, s0 = pre[(l, b, h)]
            K1, V1, p1, s1 = gpu.export_slab(l, b, h)
            idx = torch.from_numpy(kept[b])
            assert K1.shape[0] == sl.n == len(kept[b])
            assert torch.equal(p1, p0[idx]) and torch.equal(H.bits(s1), H.bits(s0[idx]))
            assert torch.equal(H.bits(K1), H.bits(K0[idx])) and torch.equal(H.bits(V1), H.bits(V0[idx]))
            assert np.array_equal(p1.numpy(), sl.pos[:sl.n])
            sl.score[:sl.n] = s1.numpy().astype(np.float64)       # re-synchronise
        if n_before > cfg.budget:
            events += 1
            moved += sum(int((kk != np.arange(len(kk))).sum()) for kk in kept)
    assert events >= 3 and moved > 0 and worst_score <= H.TOL_DELTA, (events, moved, worst_score)
    assert worst_key <= 1e-4 * cfg.layers * cfg.kv_heads, worst_key
    gpu.close()
