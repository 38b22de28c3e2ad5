"""Pins for the oracle's schedule and cost helpers: the paper's closed forms and printed values."""
import os

import numpy as np

from oracle import dynts_oracle as O
import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def load_golden():
    vals = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if "=" in line:
                k, v = line.split("=", 1)
                vals[k.strip()] = v.strip()
    return vals


def test_break_even_example_from_paper():
    g = load_golden()
    d, L = int(g["break_even_example_d"]), int(g["break_even_example_L"])
    rhs = int(g["break_even_example_rhs"])
    assert 1.5 * d / L == rhs                                  # the approximation the paper prints
    exact = O.break_even_volume(d, L, 1)
    assert rhs <= exact < rhs + 0.01                           # (6d^2+d)/(4Ld) = 1.5 d/L + 1/(4L)
    K = int(g["break_even_example_K"])
    assert K >= exact and O.computational_gain(L, d, K, 1) > 0
    assert O.computational_gain(L, d, rhs, 1) < 0 < O.computational_gain(L, d, rhs + 1, 1)


def test_predictor_flops_and_dims():
    g = load_golden()
    for key in ("predictor_dims_qwen", "predictor_dims_llama"):
        d, m1, m2, m3 = [int(x) for x in g[key].split()]
        assert (m1, m2, m3) == (2 * d, d // 2, 1)
        assert O.predictor_flops(d) == 2 * (d * m1 + m1 * m2 + m2 * m3) == 6 * d * d + d


def test_attention_flops_linear_in_length():
    assert O.attn_flops(32, 4096, 1) == 4 * 32 * 4096
    assert O.attn_flops(32, 4096, 2048) - O.attn_flops(32, 4096, 2048 - 900) == 4 * 32 * 4096 * 900


def test_kv_length_ratio_example():
    g = load_golden()
    assert round(int(g["kv_length_full"]) / int(g["kv_length_dynts"]), 1) == float(g["kv_length_ratio"])


def test_eviction_count_formula_cases():
    # below the budget nothing has fired; at the budget the first event fires
    assert O.eviction_count(32, 10, 160, 32) == 0
    assert O.eviction_count(32, 127, 160, 32) == 0
    assert O.eviction_count(32, 128, 160, 32) == 1
    assert O.effective_length(32, 128, 160, 32) == 128
    assert O.effective_length(32, 159, 160, 32) == 159
    assert O.effective_length(32, 160, 160, 32) == 128


def _lengths(cfg, steps):
    cache = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, cfg.capacity)
    pk, pv = W.prompt_kv(cfg, 11)
    events = []
    lengths = O.run_schedule(cache, pk, pv, W.DecodeStream(cfg, 11), steps, cfg.budget, cfg.evict_interval,
                             on_evict=lambda s, kept: events.append((s, len(kept[0][0][0]))))
    return cache, lengths, events


def test_config1_lengths_follow_closed_form():
    """'Every E steps down to B' is the paper's 'fire at the budget, evict K' with the paper's
    budget = B + E and K = E: the oracle's length after step i must equal S_i."""
    cfg = W.get_config("c1_tiny_fp32")
    cache, lengths, events = _lengths(cfg, cfg.decode_steps)
    B_paper, K = cfg.budget + cfg.evict_interval, cfg.evict_interval
    for i, n in enumerate(lengths, start=1):
        assert n == O.effective_length(cfg.prompt, i, B_paper, K), i
    assert max(lengths) <= cfg.budget + cfg.evict_interval - 1
    nontrivial = [s for s, m in events if s >= cfg.budget + cfg.evict_interval - cfg.prompt]
    assert len(nontrivial) == 13 == O.eviction_count(cfg.prompt, cfg.decode_steps, B_paper, K)
    s = cache.slab(0, 0, 0)
    assert list(s.pos[:cfg.prompt]) == list(range(cfg.prompt))          # question window kept
    assert list(s.pos[s.n - cfg.window:s.n]) == list(range(cfg.prompt + cfg.decode_steps - cfg.window,
                                                           cfg.prompt + cfg.decode_steps))


def test_shortened_config2_shape_schedule():
    cfg = W.get_config("c2_llama8b").scaled(layers=1, kv_heads=2, q_heads=8, prompt=16, budget=64,
                                             window=8, evict_interval=8, decode_steps=120)
    cache, lengths, _ = _lengths(cfg, cfg.decode_steps)
    for i, n in enumerate(lengths, start=1):
        assert n == O.effective_length(cfg.prompt, i, cfg.budget + cfg.evict_interval, cfg.evict_interval)


def test_planted_keys_attract_mass():
    """Sanity of the input recipe (not of the method): planted keys get most of the mass."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, prompt=8, decode_steps=0)
    u = W.gen._unit_dirs(cfg, 5)
    k, _ = W.prompt_kv(cfg, 5, n_tokens=400)
    q, _, _ = W.DecodeStream(cfg, 5).step(1)
    a = O.attention_weights(q[0, 0, 0:4], k[0, 0, 0])
    proj = k[0, 0, 0] @ u[0, 0, 0]
    crit = proj > 3.0
    assert 0.02 < crit.mean() < 0.09
    assert a[:, crit].sum() / a.sum() > 0.5
