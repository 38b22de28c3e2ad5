"""Float64 CPU oracle for budget-limited decode attention, importance accumulation and eviction.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the hot path
computes.  It shares no code with the CUDA library and must never be imported by the product
package; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.

What each function follows in the paper:

* ``attention_weights`` / ``decode_step`` -- token-level attention of the decode query over the
  retained cache, Eq. 4 (softmax of q.k/sqrt(d_k) over every cached position, the new one
  included) and Eq. 5 (weighted sum of values).
* ``decode_step`` (delta/score part) -- Eq. 6: a token's importance is the attention it receives
  summed over query rows.  Here the rows are the decode queries seen so far, summed over the
  query heads that share the KV head (Appendix B.1 aggregates heads; sum is the reading taken here).
* ``prefill_attention`` -- the same Eq. 4-5 for every prompt position (the prefill phase that fills
  the question window of Section 4.2).
* ``select_keep`` / ``evict`` -- Section 4.2: the question window (the first M rows) and the local
  window (the last W rows) are always retained, the top-k of the selection window by score are
  retained, the rest are evicted.  Ties go to the lower index; retained rows keep their order.
* ``aggregate_scores`` / ``evict_global`` -- Appendix B.1's aggregation of the importance across all
  layers and heads, used online: one selection per sequence shared by every slab.
* ``set_new_scores`` / ``predictor_mlp`` / ``paper_target`` / ``run_paper_schedule`` -- Section 4.1
  (Eq. 7: one predictor score per token) and Section 4.2 as written (select when the count reaches
  the budget B, keep a ratio of the selection window).
* ``fp8_e4m3_*`` / ``OracleCache(kv_format="e4m3")`` -- no passage of the paper: K/V rows stored as
  8-bit floats (the OCP 8-bit floating point format E4M3: 1 sign, 4 exponent bits with bias 7,
  3 mantissa bits, no infinities, largest finite value 448) with one scale per tensor.  A row is
  stored as the nearest representable value of x / scale (ties to the even code, saturating) and
  read back as value * scale; everything downstream is unchanged.
* ``eviction_count`` / ``effective_length`` -- Section 5, the closed form for the cache length.
* ``attn_flops`` / ``predictor_flops`` / ``break_even_volume`` -- Appendix A and Eq. 9-10.

Pinned by tests/test_oracle_*.py against a library attention routine, closed forms, brute-force
ranking and the values the paper prints.  Parity unpinned: the synthetic "planted critical key"
input recipe (it is an input distribution, not part of the method).
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np


# ----------------------------------------------------------------------------------------------
# Eq. 4-5: attention of one query head over n cached rows
# ----------------------------------------------------------------------------------------------

def attention_weights(q: np.ndarray, K: np.ndarray) -> np.ndarray:
    """alpha_j = exp(e_j) / sum_i exp(e_i), e_j = q.k_j / sqrt(d_k)   (Eq. 4).

    q: [G, d] query heads of one group, K: [n, d].  Returns alpha [G, n] in float64.
    The row maximum is subtracted before exponentiation; this leaves Eq. 4 unchanged.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    d_k = K.shape[1]
    e = (q @ K.T) / math.sqrt(d_k)
    e = e - e.max(axis=1, keepdims=True)
    p = np.exp(e)
    return p / p.sum(axis=1, keepdims=True)


def attention_output(alpha: np.ndarray, V: np.ndarray) -> np.ndarray:
    """o = sum_j alpha_j v_j   (Eq. 5).  alpha [G, n], V [n, d] -> [G, d]."""
    return alpha @ np.asarray(V, dtype=np.float64)


# ----------------------------------------------------------------------------------------------
# 8-bit K/V storage (E4M3): the format written out from its definition
# ----------------------------------------------------------------------------------------------

def fp8_e4m3_values() -> np.ndarray:
    """The 127 non-negative finite E4M3 values by code 0..126 (ascending): exponent field 0 holds
    the subnormals m/8 * 2^-6, fields 1..15 hold (1 + m/8) * 2^(e - 7); code 127 (all ones) is NaN."""
    vals = []
    for code in range(127):
        e, m = code >> 3, code & 7
        vals.append(m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(vals, dtype=np.float64)


def fp8_e4m3_encode(x: np.ndarray) -> np.ndarray:
    """Codes (uint8, sign in bit 7) of the E4M3 values nearest to x: round to nearest, ties to the
    code with an even mantissa bit, magnitudes beyond 448 saturate to 448.  x is taken as float32
    (the precision the device converts from)."""
    x = np.asarray(x, dtype=np.float32).astype(np.float64)
    table = fp8_e4m3_values()
    a = np.abs(x)
    hi = np.clip(np.searchsorted(table, a, side="left"), 0, 126)      # first value >= a (or the last)
    lo = np.clip(hi - 1, 0, 126)
    d_lo, d_hi = a - table[lo], table[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo)
    code = np.where(a >= table[126], 126, code)
    return (code | np.where(np.signbit(x), 128, 0)).astype(np.uint8)


def fp8_e4m3_decode(code: np.ndarray) -> np.ndarray:
    code = np.asarray(code, dtype=np.uint8)
    mag = fp8_e4m3_values()[np.minimum(code & 127, 126)]
    return np.where(code & 128, -mag, mag)


def fp8_e4m3_store(x: np.ndarray, scale: float) -> np.ndarray:
    """What a cache with E4M3 rows holds for x: decode(encode(x / scale)) * scale, the division in
    float32 (the precision in which the device takes this integer decision)."""
    x32 = np.asarray(x, dtype=np.float32) / np.float32(scale)
    return fp8_e4m3_decode(fp8_e4m3_encode(x32)) * float(np.float32(scale))


# ----------------------------------------------------------------------------------------------
# Cache state
# ----------------------------------------------------------------------------------------------

class Slab:
    """Retained rows of one (layer, sequence, KV head): K, V, original positions and scores."""

    __slots__ = ("K", "V", "pos", "score", "n")

    def __init__(self, capacity: int, d: int):
        self.K = np.zeros((capacity, d), dtype=np.float64)
        self.V = np.zeros((capacity, d), dtype=np.float64)
        self.pos = np.zeros(capacity, dtype=np.int64)
        self.score = np.zeros(capacity, dtype=np.float64)
        self.n = 0


class OracleCache:
    def __init__(self, layers: int, batch: int, q_heads: int, kv_heads: int, head_dim: int,
                 window: int, capacity: int, kv_format: Optional[str] = None, k_scale: float = 1.0,
                 v_scale: float = 1.0):
        assert q_heads % kv_heads == 0
        assert kv_format in (None, "e4m3")
        self.kv_format, self.k_scale, self.v_scale = kv_format, k_scale, v_scale
        self.layers, self.batch = layers, batch
        self.q_heads, self.kv_heads, self.head_dim = q_heads, kv_heads, head_dim
        self.group = q_heads // kv_heads
        self.window = window
        self.capacity = capacity
        self._slabs = {}                 # (layer, seq, head) -> Slab, storage created on first use
        self.n_pinned = [0] * batch      # M: question rows, immune to eviction
        self.next_pos = [0] * batch      # position id given to the next appended token

    def slab(self, layer: int, seq: int, head: int) -> Slab:
        key = (layer, seq, head)
        s = self._slabs.get(key)
        if s is None:
            s = self._slabs[key] = Slab(self.capacity, self.head_dim)
        return s

    def stored_k(self, k: np.ndarray) -> np.ndarray:
        """The value the cache holds for a key row (the row itself unless rows are 8-bit)."""
        return fp8_e4m3_store(k, self.k_scale) if self.kv_format == "e4m3" else k

    def stored_v(self, v: np.ndarray) -> np.ndarray:
        return fp8_e4m3_store(v, self.v_scale) if self.kv_format == "e4m3" else v

    def length(self, seq: int) -> int:
        return self.slab(0, seq, 0).n

    def units(self):
        for l in range(self.layers):
            for b in range(self.batch):
                for h in range(self.kv_heads):
                    yield l, b, h, self.slab(l, b, h)


def prefill(cache: OracleCache, k: np.ndarray, v: np.ndarray, n_pinned: Optional[int] = None,
            seq: Optional[int] = None) -> None:
    """Load prompt rows.  k, v: [L, Nb, Hkv, T, d] (or [L, Hkv, T, d] with ``seq`` given).

    The first ``n_pinned`` rows (default: all T) are the question window; they get score +inf
    (Section 4.2) and are never evicted.  The remaining rows start with score 0.
    """
    seqs = range(cache.batch) if seq is None else [seq]
    for b in seqs:
        T = k.shape[-2]
        m = T if n_pinned is None else n_pinned
        assert 0 <= m <= T <= cache.capacity
        for l in range(cache.layers):
            for h in range(cache.kv_heads):
                s = cache.slab(l, b, h)
                src_k = k[l, b, h] if seq is None else k[l, h]
                src_v = v[l, b, h] if seq is None else v[l, h]
                s.K[:T] = cache.stored_k(src_k)
                s.V[:T] = cache.stored_v(src_v)
                s.pos[:T] = np.arange(T)
                s.score[:T] = 0.0
                s.score[:m] = np.inf
                s.n = T
        cache.n_pinned[b] = m
        cache.next_pos[b] = T


def decode_step(cache: OracleCache, q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                active: Optional[Sequence[bool]] = None, accumulate: bool = True):
    """One decode step for every (layer, sequence, KV head).

    q [L, Nb, Hq, d]; k_new, v_new [L, Nb, Hkv, d].  For each slab: append the new row (its
    score starts at 0), attend over all n rows including the new one (Eq. 4-5), add each row's
    attention mass summed over the group's query heads to its score (Eq. 6).

    With ``accumulate=False`` the scores are left alone (the new row's score stays 0): the
    caller supplies them, as the paper does with its Importance Predictor (Section 4.1, Eq. 7).

    Returns (out [L, Nb, Hq, d] float64, delta) where delta[l][b][h] is this step's mass per
    row, an array of length n.
    """
    L, Nb, Hkv, G, d = cache.layers, cache.batch, cache.kv_heads, cache.group, cache.head_dim
    out = np.zeros((L, Nb, cache.q_heads, d), dtype=np.float64)
    delta = [[[None] * Hkv for _ in range(Nb)] for _ in range(L)]
    for l, b, h, s in cache.units():
        if active is not None and not active[b]:
            continue
        assert s.n < cache.capacity, "append past capacity: an eviction was skipped"
        s.K[s.n] = cache.stored_k(k_new[l, b, h])
        s.V[s.n] = cache.stored_v(v_new[l, b, h])
        s.pos[s.n] = cache.next_pos[b]
        s.score[s.n] = 0.0
        s.n += 1
        n = s.n
        qg = q[l, b, h * G:(h + 1) * G]
        alpha = attention_weights(qg, s.K[:n])                 # Eq. 4
        out[l, b, h * G:(h + 1) * G] = attention_output(alpha, s.V[:n])   # Eq. 5
        dl = alpha.sum(axis=0)                                 # Eq. 6, one more query row per head
        if accumulate:                                         # else: scores come from outside (Eq. 7)
            s.score[:n] += dl
        delta[l][b][h] = dl
    for b in range(Nb):
        if active is None or active[b]:
            cache.next_pos[b] += 1
    return out, delta


# ----------------------------------------------------------------------------------------------
# Eq. 4-5 over the prompt: the prefill phase that fills the question window (Section 4.2)
# ----------------------------------------------------------------------------------------------

def prefill_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Token-level attention of every prompt position over the positions up to and including
    itself (Eq. 4-5 with t = 1..M), for all layers, sequences and heads.

    q [L, Nb, Hq, T, d]; k, v [L, Nb, Hkv, T, d] -> out [L, Nb, Hq, T, d] float64.  Query head g
    of KV head h is head h * G + g (the grouping of decode_step)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    L, Nb, Hq, T, d = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    out = np.zeros_like(q)
    for l in range(L):
        for b in range(Nb):
            for hq in range(Hq):
                h = hq // G
                for t in range(T):
                    alpha = attention_weights(q[l, b, hq, t][None, :], k[l, b, h, :t + 1])   # Eq. 4 over j <= t
                    out[l, b, hq, t] = attention_output(alpha, v[l, b, h, :t + 1])[0]       # Eq. 5
    return out


# ----------------------------------------------------------------------------------------------
# Section 4.2: budgeted selection
# ----------------------------------------------------------------------------------------------

def select_keep(score32: np.ndarray, n: int, n_pinned: int, window: int, target: int) -> np.ndarray:
    """Indices (ascending) of the rows that survive an eviction down to ``target`` rows.

    Rows [0, n_pinned) (question window) and [n - window, n) (local window) always survive.
    Of the selection window [n_pinned, n - window) the k = target - n_pinned - window rows with
    the highest score survive; equal scores are ranked by lower index first.  Scores are
    compared as float32 values (the precision the scores are stored in on the device).
    If n <= target nothing is evicted.
    """
    if n <= target:
        return np.arange(n, dtype=np.int64)
    k = target - n_pinned - window
    if k < 0:
        raise ValueError("question window + local window exceed the target length")
    lo, hi = n_pinned, n - window
    sc = np.asarray(score32[:n], dtype=np.float32)
    ranked = sorted(range(lo, hi), key=lambda j: (-float(sc[j]), j))
    kept = list(range(0, lo)) + sorted(ranked[:k]) + list(range(hi, n))
    return np.asarray(kept, dtype=np.int64)


def evict(cache: OracleCache, target, scores32=None):
    """Evict every slab down to ``target`` rows (an int, or one int per sequence).

    ``scores32(l, b, h)`` may supply the float32 score array the decision is taken from (used to
    replay the device's decisions from the device's own scores); by default the slab's own
    score, rounded to float32, decides.  Survivors are gathered in ascending index order into
    rows [0, target); K, V, pos and score move together.

    Returns kept[l][b][h] = the surviving row indices (before compaction).
    """
    L, Nb, Hkv = cache.layers, cache.batch, cache.kv_heads
    kept_all = [[[None] * Hkv for _ in range(Nb)] for _ in range(L)]
    for l, b, h, s in cache.units():
        tgt = int(target if np.isscalar(target) else target[b])
        sc = s.score[:s.n].astype(np.float32) if scores32 is None else scores32(l, b, h)
        kept = select_keep(sc, s.n, cache.n_pinned[b], cache.window, tgt)
        m = len(kept)
        s.K[:m] = s.K[kept]
        s.V[:m] = s.V[kept]
        s.pos[:m] = s.pos[kept]
        s.score[:m] = s.score[kept]
        s.n = m
        kept_all[l][b][h] = kept
    return kept_all


# ----------------------------------------------------------------------------------------------
# Appendix B.1: one importance score per token, aggregated across all layers and heads
# ----------------------------------------------------------------------------------------------

def aggregate_scores(cache: OracleCache, seq: int) -> np.ndarray:
    """Appendix B.1 aggregates the attention a token receives across all layers and heads into one
    importance score per token.  Online form: agg[j] = sum over every layer l and KV head h of
    score[l][seq][h][j] (all slabs of a sequence must hold the same tokens).  Plain float64 sum;
    pinned rows (+inf) stay +inf."""
    n = cache.length(seq)
    agg = np.zeros(n, dtype=np.float64)
    for l in range(cache.layers):
        for h in range(cache.kv_heads):
            s = cache.slab(l, seq, h)
            assert s.n == n, "slabs of one sequence differ in length"
            agg += s.score[:n]
    return agg


def evict_global(cache: OracleCache, target, keys32=None):
    """Section 4.2's selection taken once per sequence on the aggregated score and applied to every
    layer and KV head: all slabs of a sequence keep the same rows.  ``keys32(b)`` may supply the
    float32 array the decision for sequence b is taken from (used to replay the device's decisions
    from the device's own aggregated scores); by default the float64 aggregate, rounded once to
    float32, decides.  Returns kept[b]."""
    kept_all = []
    for b in range(cache.batch):
        tgt = int(target if np.isscalar(target) else target[b])
        n = cache.length(b)
        keys = aggregate_scores(cache, b).astype(np.float32) if keys32 is None else np.asarray(keys32(b)[:n], dtype=np.float32)
        kept = select_keep(keys, n, cache.n_pinned[b], cache.window, tgt)
        m = len(kept)
        for l in range(cache.layers):
            for h in range(cache.kv_heads):
                s = cache.slab(l, b, h)
                s.K[:m] = s.K[kept]
                s.V[:m] = s.V[kept]
                s.pos[:m] = s.pos[kept]
                s.score[:m] = s.score[kept]
                s.n = m
        kept_all.append(kept)
    return kept_all


# ----------------------------------------------------------------------------------------------
# Section 4.1-4.2: predictor scores and the paper's own trigger
# ----------------------------------------------------------------------------------------------

def set_new_scores(cache: OracleCache, s_new: Sequence[float], active: Optional[Sequence[bool]] = None) -> None:
    """Section 4.2: a newly generated token's importance score is appended beside its KV.  The
    paper's predictor emits one scalar per token (Eq. 7), so the row appended by the latest
    decode step gets the same score s_new[b] in every layer and KV head of sequence b."""
    for l, b, h, s in cache.units():
        if active is not None and not active[b]:
            continue
        assert s.n > 0
        s.score[s.n - 1] = np.float32(s_new[b])


def predictor_mlp(h: np.ndarray, W1, b1, W2, b2, W3, b3, activation: str = "none") -> np.ndarray:
    """Importance Predictor head (Section 4.1, Appendix A): a three-layer MLP d -> 2d -> d/2 -> 1 on
    the final hidden state h [Nb, d]; returns one score per sequence, float64.  W_i is [out, in].
    The paper calls the layers linear and names no activation; ``activation`` ("none" or "relu",
    applied after the first two layers) is a parameter of this library."""
    act = (lambda x: x) if activation == "none" else (lambda x: np.maximum(x, 0.0))
    x = np.asarray(h, dtype=np.float64)
    y1 = act(x @ np.asarray(W1, dtype=np.float64).T + np.asarray(b1, dtype=np.float64))
    y2 = act(y1 @ np.asarray(W2, dtype=np.float64).T + np.asarray(b2, dtype=np.float64))
    y3 = y2 @ np.asarray(W3, dtype=np.float64).T + np.asarray(b3, dtype=np.float64)
    return y3.reshape(-1)


def paper_target(M: int, B: int, W_l: int, ratio: float) -> int:
    """Rows kept by one selection of Section 4.2: the question window (M rows), the local window
    (W_l rows) and the top ratio * W_s rows of the selection window, W_s = B - M - W_l.  The paper
    does not say how ratio * W_s is rounded; it is rounded down here."""
    W_s = B - M - W_l
    if W_s < 0:
        raise ValueError("question window + local window exceed the budget")
    return M + int(math.floor(ratio * W_s)) + W_l


def run_paper_schedule(cache: OracleCache, prompt_k, prompt_v, stream, steps: int, B: int, ratio: float,
                       new_scores=None, on_evict=None) -> List[int]:
    """Section 4.2 as written: prefill (question pinned), decode; once the row count reaches the
    budget B, select down to paper_target(...).  ``new_scores(s)`` -> [Nb] gives the predictor
    scores of step s (then attention mass is not accumulated); None => Eq. 6 mass accumulates.
    Returns the cache length after each step."""
    prefill(cache, prompt_k, prompt_v)
    M = cache.n_pinned[0]
    lengths = []
    for s in range(1, steps + 1):
        q, k_new, v_new = stream.step(s)
        decode_step(cache, q, k_new, v_new, accumulate=new_scores is None)
        if new_scores is not None:
            set_new_scores(cache, new_scores(s))
        if cache.length(0) >= B:
            kept = evict(cache, paper_target(M, B, cache.window, ratio))
            if on_evict is not None:
                on_evict(s, kept)
        lengths.append(cache.length(0))
    return lengths


# ----------------------------------------------------------------------------------------------
# Section 5 / Appendix A: closed forms
# ----------------------------------------------------------------------------------------------

def eviction_count(M: int, i: int, B: int, K: int) -> int:
    """n_i = max(0, floor(((M + i) - B) / K) + 1): eviction events up to decode step i."""
    return max(0, (M + i - B) // K + 1)


def effective_length(M: int, i: int, B: int, K: int) -> int:
    """S_i = M + i - n_i * K: cache length at decode step i when K rows leave at each event."""
    return M + i - eviction_count(M, i, B, K) * K


def attn_flops(L: int, d: int, S: int) -> int:
    """Attention cost of one decode step over a cache of S rows: 4 * L * d * S (Appendix A)."""
    return 4 * L * d * S


def predictor_flops(d: int) -> int:
    """MLP d -> 2d -> d/2 -> 1: 2*(d*2d + 2d*d/2 + d/2*1) = 6 d^2 + d (Appendix A)."""
    return 2 * (d * (2 * d) + (2 * d) * (d // 2) + (d // 2) * 1)


def computational_gain(L: int, d: int, K: int, n_i: int) -> int:
    """Delta C(i) = n_i * 4 L d K - (6 d^2 + d)   (Eq. 9)."""
    return n_i * 4 * L * d * K - predictor_flops(d)


def break_even_volume(d: int, L: int, n_i: int = 1) -> float:
    """Smallest eviction volume with a net gain: (6 d^2 + d) / (n_i * 4 L d)   (Eq. 10)."""
    return predictor_flops(d) / (n_i * 4 * L * d)


# ----------------------------------------------------------------------------------------------
# Schedule driver (prefill, then decode with an eviction every E steps)
# ----------------------------------------------------------------------------------------------

def run_schedule(cache: OracleCache, prompt_k, prompt_v, stream, steps: int, budget: int,
                 evict_interval: int, on_step=None, on_evict=None) -> List[int]:
    """Prefill (all prompt rows pinned), then ``steps`` decode steps; after every
    ``evict_interval``-th step evict down to ``budget``.  Returns the cache length after each
    step (after that step's eviction, if any)."""
    prefill(cache, prompt_k, prompt_v)
    lengths = []
    for s in range(1, steps + 1):
        q, k_new, v_new = stream.step(s)
        out, delta = decode_step(cache, q, k_new, v_new)
        if on_step is not None:
            on_step(s, out, delta)
        if s % evict_interval == 0:
            kept = evict(cache, budget)
            if on_evict is not None:
                on_evict(s, kept)
        lengths.append(cache.length(0))
    return lengths
