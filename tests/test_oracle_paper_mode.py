"""Pins of the oracle's predictor-score mode and of Section 4.2's own trigger (select when the row
count reaches the budget B, keep a ratio of the selection window), against the paper's closed
forms, brute force and algebraic special cases.  CPU only."""
import math

import numpy as np
import pytest

import workloads as W
from oracle import dynts_oracle as O


def _small_cfg(**kw):
    base = dict(layers=2, batch=2, kv_heads=2, q_heads=4, head_dim=16, prompt=12, budget=64, window=8, evict_interval=16)
    base.update(kw)
    return W.get_config("c1_tiny_fp32").scaled(**base)


def _score_stream(seed, batch):
    def f(s):
        return np.random.default_rng([seed, s]).standard_normal(batch).astype(np.float32)
    return f


@pytest.mark.parametrize("ratio", [0.3, 0.4, 0.75])
def test_lengths_follow_the_closed_form_of_section_5(ratio):
    """With the trigger at B and K rows leaving per event, the length after decode step i is
    S_i = M + i - n_i K, n_i = max(0, floor((M + i - B) / K) + 1)."""
    cfg = _small_cfg()
    B, M = 64, cfg.prompt
    W_s = B - M - cfg.window
    K = W_s - math.floor(ratio * W_s)
    assert O.paper_target(M, B, cfg.window, ratio) == B - K
    orc = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, B + 1)
    pk, pv = W.prompt_kv(cfg, 3)
    lengths = O.run_paper_schedule(orc, pk.astype(np.float64), pv.astype(np.float64), W.DecodeStream(cfg, 3), 200, B,
                                   ratio, new_scores=_score_stream(5, cfg.batch))
    for i, n in enumerate(lengths, start=1):
        assert n == O.effective_length(M, i, B, K), (i, n)
        assert n < B
    assert max(lengths) == B - 1 and O.eviction_count(M, 200, B, K) > 3


def test_predictor_scores_give_one_retained_set_per_sequence():
    """One scalar per token (Eq. 7) appended to every layer and head => every slab of a sequence
    retains the same positions, and they are the brute-force top-k of the selection window."""
    cfg = _small_cfg()
    B, ratio = 64, 0.4
    orc = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, B + 1)
    pk, pv = W.prompt_kv(cfg, 4)
    scores = _score_stream(9, cfg.batch)
    history = {b: {} for b in range(cfg.batch)}          # position -> score, kept by the test itself

    def new_scores(s):
        v = scores(s)
        for b in range(cfg.batch):
            history[b][cfg.prompt + s - 1] = float(v[b])
        return v

    events = []
    O.run_paper_schedule(orc, pk.astype(np.float64), pv.astype(np.float64), W.DecodeStream(cfg, 4), 150, B, ratio,
                         new_scores=new_scores, on_evict=lambda s, kept: events.append(s))
    assert len(events) >= 3
    for b in range(cfg.batch):
        ref = orc.slab(0, b, 0)
        for l in range(cfg.layers):
            for h in range(cfg.kv_heads):
                sl = orc.slab(l, b, h)
                assert np.array_equal(sl.pos[:sl.n], ref.pos[:ref.n])
        # scores stored beside the rows are the predictor's, question rows are +inf
        for j in range(ref.n):
            p = int(ref.pos[j])
            if p < cfg.prompt:
                assert np.isinf(ref.score[j])
            else:
                assert ref.score[j] == np.float32(history[b][p])


def test_one_selection_is_brute_force_top_k():
    r = np.random.default_rng(11)
    n, M, Wl, B, ratio = 40, 5, 6, 40, 0.5
    sc = r.standard_normal(n).astype(np.float32)
    sc[7] = sc[9] = sc[20]                               # ties go to the lower index
    tgt = O.paper_target(M, B, Wl, ratio)
    kept = O.select_keep(sc, n, M, Wl, tgt)
    k = tgt - M - Wl
    cand = list(range(M, n - Wl))
    best = sorted(cand, key=lambda j: (-sc[j], j))[:k]
    assert sorted(kept.tolist()) == sorted(list(range(M)) + best + list(range(n - Wl, n)))
    # Table 2's "T-Bottom" ablation is the same call on negated scores: the complement of the
    # top (W_s - k) when there are no ties
    sc2 = r.standard_normal(n).astype(np.float32)
    top = set(O.select_keep(sc2, n, M, Wl, tgt).tolist())
    bottom = set(O.select_keep(-sc2, n, M, Wl, n - (tgt - M - Wl)).tolist())
    assert (top & bottom) == set(range(M)) | set(range(n - Wl, n))


def test_predictor_mlp_shapes_flops_and_linear_collapse():
    d = 32
    r = np.random.default_rng(2)
    W1, b1 = r.standard_normal((2 * d, d)), r.standard_normal(2 * d)
    W2, b2 = r.standard_normal((d // 2, 2 * d)), r.standard_normal(d // 2)
    W3, b3 = r.standard_normal((1, d // 2)), r.standard_normal(1)
    h = r.standard_normal((5, d))
    # Appendix A counts 2 flops per weight: 6 d^2 + d
    assert 2 * (W1.size + W2.size + W3.size) == O.predictor_flops(d) == 6 * d * d + d
    assert O.predictor_flops(4096) == 6 * 4096 ** 2 + 4096
    # without activation three linear layers collapse into one affine map
    A = W3 @ W2 @ W1
    c = W3 @ (W2 @ b1 + b2) + b3
    np.testing.assert_allclose(O.predictor_mlp(h, W1, b1, W2, b2, W3, b3, "none"), (h @ A.T + c).reshape(-1), rtol=1e-12)
    # ReLU is the identity on non-negative pre-activations
    Wp = [np.abs(x) for x in (W1, b1, W2, b2)]
    hp = np.abs(h)
    np.testing.assert_allclose(O.predictor_mlp(hp, Wp[0], Wp[1], Wp[2], Wp[3], W3, b3, "relu"),
                               O.predictor_mlp(hp, Wp[0], Wp[1], Wp[2], Wp[3], W3, b3, "none"), rtol=1e-12)
    # and zeroes a unit whose pre-activation is negative: one hidden unit, by hand
    assert O.predictor_mlp(np.array([[1.0, 0.0]]), np.array([[-2.0, 0.0], [3.0, 0.0], [0.0, 0.0], [0.0, 0.0]]), np.zeros(4),
                           np.array([[1.0, 1.0, 0.0, 0.0]]), np.zeros(1), np.array([[2.0]]), np.array([0.5]), "relu")[0] == 6.5


def test_accumulate_off_leaves_scores_alone():
    cfg = _small_cfg(layers=1, batch=1)
    orc = O.OracleCache(1, 1, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, 80)
    pk, pv = W.prompt_kv(cfg, 6)
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64), n_pinned=4)
    st = W.DecodeStream(cfg, 6)
    before = orc.slab(0, 0, 0).score[:12].copy()
    out_a, delta = O.decode_step(orc, *[x.astype(np.float64) for x in st.step(1)], accumulate=False)
    sl = orc.slab(0, 0, 0)
    assert np.array_equal(sl.score[:12], before) and sl.score[12] == 0.0 and sl.n == 13
    assert abs(delta[0][0][0].sum() - cfg.group) < 1e-12       # the attention itself is unchanged
    O.set_new_scores(orc, [0.25])
    assert sl.score[12] == np.float32(0.25)


def _decoded_cache(cfg, seed, steps, n_pinned=None, cap=80):
    orc = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, cap)
    pk, pv = W.prompt_kv(cfg, seed)
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64), n_pinned=n_pinned)
    st = W.DecodeStream(cfg, seed)
    for s in range(1, steps + 1):
        O.decode_step(orc, *[x.astype(np.float64) for x in st.step(s)])
    return orc


def test_aggregated_mass_is_conserved_across_layers_and_heads():
    """Appendix B.1 / Eq. 6: every decode step hands out a mass of 1 per query head, so with no
    pinned row and no eviction the aggregate over all layers and heads sums to
    layers x q_heads x steps.  A dropped layer or head breaks the total."""
    cfg = _small_cfg(layers=3, batch=2, kv_heads=2, q_heads=4)
    steps = 25
    orc = _decoded_cache(cfg, 8, steps, n_pinned=0)
    for b in range(cfg.batch):
        agg = O.aggregate_scores(orc, b)
        assert agg.dtype == np.float64 and agg.shape == (cfg.prompt + steps,)
        assert np.all(agg >= 0)
        assert abs(agg.sum() - cfg.layers * cfg.q_heads * steps) < 1e-9
        # the row appended by the last step has been attended to once, by every head of every layer
        assert 0 < agg[-1] <= cfg.layers * cfg.q_heads


def test_aggregate_of_hand_set_scores_has_the_closed_form_and_ignores_slab_order():
    """score[l][h][j] = 10 (l + 1) + h + j / 2 has the aggregate
    Hkv * 10 * L (L + 1) / 2 + L * Hkv (Hkv - 1) / 2 + L * Hkv * j / 2; it equals the library sum over
    the stacked slabs and does not change when layers and heads are permuted."""
    L, Hkv, n = 3, 2, 20
    cfg = _small_cfg(layers=L, batch=1, kv_heads=Hkv, q_heads=4)
    orc = _decoded_cache(cfg, 11, n - cfg.prompt, n_pinned=0)
    j = np.arange(n, dtype=np.float64)
    for l in range(L):
        for h in range(Hkv):
            orc.slab(l, 0, h).score[:n] = 10.0 * (l + 1) + h + j / 2
    expect = Hkv * 10.0 * L * (L + 1) / 2 + L * Hkv * (Hkv - 1) / 2 + L * Hkv * j / 2
    agg = O.aggregate_scores(orc, 0)
    assert np.array_equal(agg, expect)
    stacked = np.stack([orc.slab(l, 0, h).score[:n] for l in range(L) for h in range(Hkv)])
    assert np.array_equal(agg, stacked.sum(axis=0))
    perm = np.random.default_rng(3).permutation(L * Hkv)
    rows = stacked[perm]
    for i, (l, h) in enumerate((l, h) for l in range(L) for h in range(Hkv)):
        orc.slab(l, 0, h).score[:n] = rows[i]
    assert np.array_equal(O.aggregate_scores(orc, 0), expect)
    # one pinned row in one slab pins the token's aggregate
    orc.slab(1, 0, 1).score[4] = np.inf
    assert O.aggregate_scores(orc, 0)[4] == np.inf


def test_global_selection_shares_one_retained_set_and_matches_brute_force():
    cfg = _small_cfg(layers=3, batch=2, kv_heads=2, q_heads=4)
    orc = _decoded_cache(cfg, 8, 40)
    n = orc.length(0)
    # brute force on the float64 aggregate: rank the selection window by (sum descending, index)
    expect = []
    for b in range(cfg.batch):
        tot = np.stack([orc.slab(l, b, h).score[:n] for l in range(cfg.layers) for h in range(cfg.kv_heads)]).sum(axis=0)
        cand = list(range(cfg.prompt, n - cfg.window))
        gaps = np.diff(np.sort(tot[cand]))
        assert gaps.min() > 1e-4 * tot[cand].max()       # well separated: rounding to float32 cannot reorder them
        k = 40 - cfg.prompt - cfg.window
        best = sorted(sorted(cand, key=lambda j: (-tot[j], j))[:k])
        expect.append(list(range(cfg.prompt)) + best + list(range(n - cfg.window, n)))
    pos_before = {b: orc.slab(0, b, 0).pos[:n].copy() for b in range(cfg.batch)}
    kept = O.evict_global(orc, 40)
    for b in range(cfg.batch):
        assert kept[b].tolist() == expect[b]
        for l in range(cfg.layers):
            for h in range(cfg.kv_heads):
                sl = orc.slab(l, b, h)
                assert sl.n == 40 and np.array_equal(sl.pos[:40], pos_before[b][kept[b]])


def test_global_selection_sees_every_slab_and_takes_supplied_keys():
    """A row that only ONE slab rates highly (by a margin above all other sums) must survive in all
    slabs; keys handed in replace the aggregate."""
    cfg = _small_cfg(layers=3, batch=1, kv_heads=2, q_heads=4)
    for (l, h) in [(0, 0), (2, 1), (1, 0)]:
        orc = _decoded_cache(cfg, 13, 40)
        n = orc.length(0)
        cand = np.arange(cfg.prompt, n - cfg.window)
        low = cand[np.argmin(O.aggregate_scores(orc, 0)[cand])]      # would be evicted first ...
        kept0 = O.evict_global(_decoded_cache(cfg, 13, 40), 40)[0]
        assert low not in kept0
        orc.slab(l, 0, h).score[low] += 1e6                           # ... unless this one slab says otherwise
        kept = O.evict_global(orc, 40)[0]
        assert low in kept
    orc = _decoded_cache(cfg, 13, 40)
    n = orc.length(0)
    keys = np.arange(n, dtype=np.float32)                             # supplied keys: later rows rank higher
    kept = O.evict_global(orc, 40, keys32=lambda b: keys)[0]
    k = 40 - cfg.prompt - cfg.window
    assert kept.tolist() == list(range(cfg.prompt)) + list(range(n - cfg.window - k, n))


def test_global_selection_with_one_slab_is_the_per_slab_selection():
    cfg = _small_cfg(layers=1, batch=1, kv_heads=1, q_heads=2)
    a = O.OracleCache(1, 1, 2, 1, cfg.head_dim, cfg.window, 80)
    b = O.OracleCache(1, 1, 2, 1, cfg.head_dim, cfg.window, 80)
    pk, pv = W.prompt_kv(cfg, 9)
    for c in (a, b):
        O.prefill(c, pk.astype(np.float64), pv.astype(np.float64))
    st = W.DecodeStream(cfg, 9)
    for s in range(1, 31):
        x = [t.astype(np.float64) for t in st.step(s)]
        O.decode_step(a, *x)
        O.decode_step(b, *x)
    ka = O.evict(a, 30)[0][0][0]
    kb = O.evict_global(b, 30)[0]
    assert np.array_equal(ka, kb) and np.array_equal(a.slab(0, 0, 0).K[:30], b.slab(0, 0, 0).K[:30])
