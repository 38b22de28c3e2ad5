"""Pins for the oracle's attention and importance accumulation (Eq. 4-6).

Each test checks the oracle against something fixed outside it: a library attention routine,
a closed form, an invariant of softmax, or a pure-Python loop on a tiny case.
"""
import math

import numpy as np
import pytest
import torch

from oracle import dynts_oracle as O


def _fresh(L=2, Nb=2, Hq=4, Hkv=2, d=16, W=2, cap=64):
    return O.OracleCache(L, Nb, Hq, Hkv, d, W, cap)


def _rand_step(rng, c):
    q = rng.standard_normal((c.layers, c.batch, c.q_heads, c.head_dim))
    k = rng.standard_normal((c.layers, c.batch, c.kv_heads, c.head_dim))
    v = rng.standard_normal((c.layers, c.batch, c.kv_heads, c.head_dim))
    return q, k, v


def test_full_cache_equals_library_attention():
    """Budget >= length: the oracle must equal textbook softmax attention.  The library routine
    (torch SDPA, float64, CPU) gets K/V with each KV head repeated for its query group."""
    rng = np.random.default_rng(0)
    c = _fresh(L=2, Nb=2, Hq=6, Hkv=2, d=32, cap=40)
    T = 9
    pk = rng.standard_normal((2, 2, 2, T, 32))
    pv = rng.standard_normal((2, 2, 2, T, 32))
    O.prefill(c, pk, pv)
    hist_k, hist_v = [pk], [pv]
    for _ in range(12):
        q, k, v = _rand_step(rng, c)
        out, _ = O.decode_step(c, q, k, v)
        hist_k.append(k[:, :, :, None, :])
        hist_v.append(v[:, :, :, None, :])
        K = torch.from_numpy(np.concatenate(hist_k, axis=3))   # [L, Nb, Hkv, n, d]
        V = torch.from_numpy(np.concatenate(hist_v, axis=3))
        G = c.group
        Kr = K.repeat_interleave(G, dim=2).flatten(0, 1)       # [L*Nb, Hq, n, d]
        Vr = V.repeat_interleave(G, dim=2).flatten(0, 1)
        Q = torch.from_numpy(q).flatten(0, 1)[:, :, None, :]   # [L*Nb, Hq, 1, d]
        ref = torch.nn.functional.scaled_dot_product_attention(Q, Kr, Vr)[:, :, 0, :]
        np.testing.assert_allclose(out.reshape(ref.shape), ref.numpy(), rtol=1e-12, atol=1e-13)


def test_weights_match_library_softmax_and_column_sums():
    """alpha against scipy's softmax of einsum logits; the step's mass is alpha's column sum."""
    from scipy.special import softmax
    rng = np.random.default_rng(1)
    c = _fresh(L=1, Nb=1, Hq=4, Hkv=1, d=8, cap=16)
    for _ in range(6):
        q, k, v = _rand_step(rng, c)
        _, delta = O.decode_step(c, q, k, v)
        s = c.slab(0, 0, 0)
        logits = np.einsum("gc,nc->gn", q[0, 0], s.K[:s.n]) / math.sqrt(8)
        a = softmax(logits, axis=1)
        np.testing.assert_allclose(delta[0][0][0], a.sum(axis=0), rtol=1e-12)


def test_zero_query_gives_uniform_weights():
    """q = 0: alpha = 1/n, o = mean(V), every row's mass is G/n (closed form)."""
    rng = np.random.default_rng(2)
    c = _fresh()
    for step in range(1, 6):
        _, k, v = _rand_step(rng, c)
        q = np.zeros((c.layers, c.batch, c.q_heads, c.head_dim))
        out, delta = O.decode_step(c, q, k, v)
        for l, b, h, s in c.units():
            mean_v = s.V[:s.n].mean(axis=0)
            for g in range(c.group):
                np.testing.assert_allclose(out[l, b, h * c.group + g], mean_v, rtol=1e-13, atol=1e-15)
            np.testing.assert_allclose(delta[l][b][h], c.group / s.n, rtol=1e-13)


def test_mass_conservation():
    """Softmax rows sum to 1, so each step adds exactly G to a slab and, with no eviction, the
    scores of the unpinned rows sum to G * steps; all masses are non-negative."""
    rng = np.random.default_rng(3)
    c = _fresh()
    steps = 20
    for _ in range(steps):
        q, k, v = _rand_step(rng, c)
        _, delta = O.decode_step(c, q, k, v)
        for l, b, h, s in c.units():
            assert abs(delta[l][b][h].sum() - c.group) < 1e-12
            assert (delta[l][b][h] >= 0).all()
    for l, b, h, s in c.units():
        assert abs(s.score[:s.n].sum() - c.group * steps) < 1e-10


def test_self_attention_included_single_row():
    """With an empty cache the new token attends only to itself: alpha = 1, o = v_new."""
    rng = np.random.default_rng(4)
    c = _fresh()
    q, k, v = _rand_step(rng, c)
    out, delta = O.decode_step(c, q, k, v)
    G = c.group
    for l, b, h, s in c.units():
        assert s.n == 1
        for g in range(G):
            np.testing.assert_allclose(out[l, b, h * G + g], v[l, b, h], rtol=0, atol=0)
        np.testing.assert_allclose(delta[l][b][h], [G])


def test_dominant_logit_selects_its_value():
    """One key aligned with the query at large norm: the output tends to that row's value."""
    rng = np.random.default_rng(5)
    c = O.OracleCache(1, 1, 1, 1, 16, 0, 32)
    pk = rng.standard_normal((1, 1, 1, 10, 16)) * 0.1
    pv = rng.standard_normal((1, 1, 1, 10, 16))
    q = rng.standard_normal((1, 1, 1, 16))
    pk[0, 0, 0, 7] = 50.0 * q[0, 0, 0] / np.linalg.norm(q)
    O.prefill(c, pk, pv, n_pinned=0)
    out, delta = O.decode_step(c, q, 0.1 * rng.standard_normal((1, 1, 1, 16)), rng.standard_normal((1, 1, 1, 16)))
    np.testing.assert_allclose(out[0, 0, 0], pv[0, 0, 0, 7], atol=1e-8)
    assert delta[0][0][0][7] > 1 - 1e-8


def test_gqa_equals_mha_with_repeated_kv():
    """A group of G query heads on one KV head equals G single-head caches with equal K/V."""
    rng = np.random.default_rng(6)
    G, d = 3, 8
    gq = O.OracleCache(1, 1, G, 1, d, 0, 16)
    mh = O.OracleCache(1, 1, G, G, d, 0, 16)
    for _ in range(7):
        q = rng.standard_normal((1, 1, G, d))
        k = rng.standard_normal((1, 1, 1, d))
        v = rng.standard_normal((1, 1, 1, d))
        o1, d1 = O.decode_step(gq, q, k, v)
        o2, d2 = O.decode_step(mh, q, np.repeat(k, G, axis=2), np.repeat(v, G, axis=2))
        np.testing.assert_allclose(o1, o2, rtol=1e-13)
        np.testing.assert_allclose(d1[0][0][0], sum(d2[0][0][g] for g in range(G)), rtol=1e-13)


def test_output_invariant_under_row_permutation():
    """Eq. 4-5 are sums over rows: permuting the cached rows leaves the output unchanged and
    permutes the masses."""
    rng = np.random.default_rng(7)
    d, n = 8, 12
    K = rng.standard_normal((n, d))
    V = rng.standard_normal((n, d))
    q = rng.standard_normal((2, d))
    perm = rng.permutation(n)
    a = O.attention_weights(q, K)
    ap = O.attention_weights(q, K[perm])
    np.testing.assert_allclose(ap, a[:, perm], rtol=1e-12)
    np.testing.assert_allclose(O.attention_output(ap, V[perm]), O.attention_output(a, V), rtol=1e-12)


def test_attention_after_eviction_equals_masked_attention():
    """Attention over the compacted cache equals attention over the kept rows of the old one."""
    rng = np.random.default_rng(8)
    c = O.OracleCache(1, 1, 2, 1, 8, 3, 40)
    pk = rng.standard_normal((1, 1, 1, 4, 8))
    pv = rng.standard_normal((1, 1, 1, 4, 8))
    O.prefill(c, pk, pv)
    for _ in range(20):
        q = rng.standard_normal((1, 1, 2, 8))
        O.decode_step(c, q, rng.standard_normal((1, 1, 1, 8)), rng.standard_normal((1, 1, 1, 8)))
    s = c.slab(0, 0, 0)
    K0, V0 = s.K[:s.n].copy(), s.V[:s.n].copy()
    kept = O.evict(c, 12)[0][0][0]
    q = rng.standard_normal((2, 8))
    a_masked = O.attention_weights(q, K0[kept])
    a_comp = O.attention_weights(q, s.K[:s.n])
    np.testing.assert_array_equal(a_masked, a_comp)
    np.testing.assert_array_equal(O.attention_output(a_masked, V0[kept]), O.attention_output(a_comp, s.V[:s.n]))


def test_python_loop_restatement_tiny():
    """Scalar loops over Eq. 4-6 on a tiny case (no matmul, no vectorised softmax)."""
    rng = np.random.default_rng(9)
    G, d, n = 2, 4, 5
    K = rng.standard_normal((n, d))
    V = rng.standard_normal((n, d))
    q = rng.standard_normal((G, d))
    alpha = O.attention_weights(q, K)
    o = O.attention_output(alpha, V)
    for g in range(G):
        e = [sum(q[g][c] * K[j][c] for c in range(d)) / math.sqrt(d) for j in range(n)]
        z = sum(math.exp(x) for x in e)
        a = [math.exp(x) / z for x in e]
        for j in range(n):
            assert abs(a[j] - alpha[g, j]) < 1e-14
        for c in range(d):
            assert abs(sum(a[j] * V[j][c] for j in range(n)) - o[g, c]) < 1e-13


def test_scale_uses_head_dim():
    """The 1/sqrt(d_k) factor: two keys whose dot products with q differ by sqrt(d)*ln(3) must get
    weights in ratio 3."""
    d = 16
    q = np.zeros((1, d)); q[0, 0] = 1.0
    K = np.zeros((2, d)); K[0, 0] = math.sqrt(d) * math.log(3.0)
    a = O.attention_weights(q, K)
    assert abs(a[0, 0] / a[0, 1] - 3.0) < 1e-12


def test_pinned_rows_stay_infinite_and_new_row_starts_at_self_mass():
    rng = np.random.default_rng(10)
    c = O.OracleCache(1, 1, 2, 1, 8, 2, 16)
    O.prefill(c, rng.standard_normal((1, 1, 1, 3, 8)), rng.standard_normal((1, 1, 1, 3, 8)))
    _, delta = O.decode_step(c, rng.standard_normal((1, 1, 2, 8)), rng.standard_normal((1, 1, 1, 8)),
                             rng.standard_normal((1, 1, 1, 8)))
    s = c.slab(0, 0, 0)
    assert np.isinf(s.score[:3]).all()
    assert s.score[3] == delta[0][0][0][3]
    assert list(s.pos[:4]) == [0, 1, 2, 3]


def test_prefill_attention_against_masked_softmax_and_decode_consistency():
    """Prefill attention row t must equal (a) the textbook masked softmax(QK^T/sqrt(d))V computed
    with a lower-triangular mask, and (b) what a decode step gives for the same token when the
    first t rows are already cached."""
    r = np.random.default_rng(12)
    L, Nb, Hq, Hkv, T, d = 2, 2, 4, 2, 9, 8
    q = r.standard_normal((L, Nb, Hq, T, d))
    k = r.standard_normal((L, Nb, Hkv, T, d))
    v = r.standard_normal((L, Nb, Hkv, T, d))
    out = O.prefill_attention(q, k, v)
    G = Hq // Hkv
    mask = np.tril(np.ones((T, T), dtype=bool))
    for l in range(L):
        for b in range(Nb):
            for hq in range(Hq):
                e = q[l, b, hq] @ k[l, b, hq // G].T / np.sqrt(d)
                e = np.where(mask, e, -np.inf)
                p = np.exp(e - e.max(axis=1, keepdims=True))
                ref = (p / p.sum(axis=1, keepdims=True)) @ v[l, b, hq // G]
                np.testing.assert_allclose(out[l, b, hq], ref, rtol=1e-12, atol=1e-12)
    # first position attends to itself only
    for hq in range(Hq):
        np.testing.assert_allclose(out[0, 0, hq, 0], v[0, 0, hq // G, 0], rtol=1e-13)
    # decode consistency: cache the first T-1 rows, decode the last token
    cache = O.OracleCache(L, Nb, Hq, Hkv, d, 2, T + 2)
    O.prefill(cache, k[..., :T - 1, :], v[..., :T - 1, :])
    o_dec, _ = O.decode_step(cache, q[..., T - 1, :], k[..., T - 1, :], v[..., T - 1, :])
    np.testing.assert_allclose(o_dec, out[..., T - 1, :], rtol=1e-12, atol=1e-12)
