"""Pins for the oracle's budgeted selection and compaction (Section 4.2)."""
import itertools

import numpy as np
import pytest

from oracle import dynts_oracle as O


def _rank_count_keep(sc, n, M, W, target):
    """Independent statement: a candidate survives iff fewer than k candidates beat it, where i
    beats j when its score is higher, or equal with i < j.  O(n^2) counting, no sort."""
    if n <= target:
        return list(range(n))
    k = target - M - W
    keep = []
    for j in range(n):
        if j < M or j >= n - W:
            keep.append(j)
            continue
        beats = 0
        for i in range(M, n - W):
            if sc[i] > sc[j] or (sc[i] == sc[j] and i < j):
                beats += 1
        if beats < k:
            keep.append(j)
    return keep


def test_exhaustive_small_alphabet_with_ties():
    """Every assignment of scores from {0, 1, 2} to n <= 7 rows, several (M, W, target)."""
    vals = np.array([0.0, 1.0, 2.0], dtype=np.float32)
    for n in range(1, 8):
        for M, W in [(0, 0), (1, 1), (2, 1), (0, 2)]:
            if M + W > n:
                continue
            for target in range(M + W, n + 1):
                for combo in itertools.product(range(3), repeat=n):
                    sc = vals[list(combo)]
                    got = list(O.select_keep(sc, n, M, W, target))
                    assert got == _rank_count_keep(sc, n, M, W, target)


def test_random_against_rank_count_and_lexsort():
    rng = np.random.default_rng(0)
    for trial in range(300):
        n = int(rng.integers(1, 60))
        M = int(rng.integers(0, n // 3 + 1))
        W = int(rng.integers(0, n // 3 + 1))
        target = int(rng.integers(M + W, n + 3))
        # coarse values give many ties
        sc = (rng.integers(0, 6, size=n) / 4.0).astype(np.float32)
        got = list(O.select_keep(sc, n, M, W, target))
        assert got == _rank_count_keep(sc, n, M, W, target)
        if n > target:
            cand = np.arange(M, n - W)
            order = cand[np.lexsort((cand, -sc[cand].astype(np.float64)))]   # library routine
            ref = sorted(list(range(M)) + list(order[: target - M - W]) + list(range(n - W, n)))
            assert got == ref


def test_invariants_count_window_pins_order():
    rng = np.random.default_rng(1)
    for trial in range(200):
        n = int(rng.integers(5, 200))
        M = int(rng.integers(0, 5))
        W = int(rng.integers(0, 5))
        target = int(rng.integers(M + W, n + 1))
        sc = rng.random(n).astype(np.float32)
        kept = O.select_keep(sc, n, M, W, target)
        assert len(kept) == min(n, target)                       # retained count <= budget
        assert (np.diff(kept) > 0).all()                         # ascending, no duplicates
        assert set(range(M)) <= set(kept)                        # question window
        assert set(range(n - W, n)) <= set(kept)                 # local window
        ev = sorted(set(range(n)) - set(kept))
        mid = [j for j in kept if M <= j < n - W]
        if ev and mid:
            assert max(sc[ev]) <= min(sc[mid])                   # nothing evicted outranks a survivor


def test_ties_prefer_lower_index():
    sc = np.zeros(10, dtype=np.float32)
    kept = O.select_keep(sc, 10, 1, 2, 6)
    assert list(kept) == [0, 1, 2, 3, 8, 9]


def test_negative_zero_ties_with_positive_zero():
    sc = np.array([0.0, -0.0, 0.0, -0.0, 5.0], dtype=np.float32)
    assert list(O.select_keep(sc, 5, 0, 0, 3)) == [0, 1, 4]


def test_special_cases():
    rng = np.random.default_rng(2)
    sc = rng.random(50).astype(np.float32)
    # budget >= length: full KV, nothing moves
    assert list(O.select_keep(sc, 50, 4, 8, 50)) == list(range(50))
    assert list(O.select_keep(sc, 50, 4, 8, 64)) == list(range(50))
    # k = 0: question + local window only (the "Window" baseline; with M = sinks it has the
    # StreamingLLM shape)
    assert list(O.select_keep(sc, 50, 4, 8, 12)) == list(range(4)) + list(range(42, 50))
    # negated scores keep the bottom-k ("T-Bottom")
    top = set(O.select_keep(sc, 50, 0, 0, 10))
    bot = set(O.select_keep(-sc, 50, 0, 0, 10))
    assert top == set(np.argsort(-sc)[:10]) and bot == set(np.argsort(sc)[:10])
    with pytest.raises(ValueError):
        O.select_keep(sc, 50, 6, 8, 12)


def test_evict_gathers_rows_bit_exactly_and_is_idempotent():
    rng = np.random.default_rng(3)
    c = O.OracleCache(2, 2, 4, 2, 8, 3, 64)
    O.prefill(c, rng.standard_normal((2, 2, 2, 5, 8)), rng.standard_normal((2, 2, 2, 5, 8)))
    for _ in range(40):
        O.decode_step(c, rng.standard_normal((2, 2, 4, 8)), rng.standard_normal((2, 2, 2, 8)),
                      rng.standard_normal((2, 2, 2, 8)))
    before = {(l, b, h): (s.K[:s.n].copy(), s.V[:s.n].copy(), s.pos[:s.n].copy(), s.score[:s.n].copy())
              for l, b, h, s in c.units()}
    kept = O.evict(c, 20)
    for l, b, h, s in c.units():
        K0, V0, p0, s0 = before[(l, b, h)]
        kk = kept[l][b][h]
        assert s.n == 20
        np.testing.assert_array_equal(s.K[:20], K0[kk])
        np.testing.assert_array_equal(s.V[:20], V0[kk])
        np.testing.assert_array_equal(s.pos[:20], p0[kk])
        np.testing.assert_array_equal(s.score[:20], s0[kk])
        assert (np.diff(s.pos[:20]) > 0).all()
        assert list(s.pos[:5]) == [0, 1, 2, 3, 4] and list(s.pos[17:20]) == [42, 43, 44]
    again = O.evict(c, 20)
    for l, b, h, s in c.units():
        assert list(again[l][b][h]) == list(range(20))


def test_external_scores_decide():
    """Scores supplied by the caller (the predictor mode) drive the same selection."""
    rng = np.random.default_rng(4)
    c = O.OracleCache(1, 1, 1, 1, 4, 2, 32)
    O.prefill(c, rng.standard_normal((1, 1, 1, 2, 4)), rng.standard_normal((1, 1, 1, 2, 4)))
    for _ in range(18):
        O.decode_step(c, rng.standard_normal((1, 1, 1, 4)), rng.standard_normal((1, 1, 1, 4)),
                      rng.standard_normal((1, 1, 1, 4)))
    ext = np.arange(20, dtype=np.float32)            # later rows score higher
    kept = O.evict(c, 10, scores32=lambda l, b, h: ext)[0][0][0]
    assert list(kept) == [0, 1] + list(range(12, 18)) + [18, 19]


def test_per_sequence_targets():
    rng = np.random.default_rng(5)
    c = O.OracleCache(1, 3, 1, 1, 4, 1, 32)
    O.prefill(c, rng.standard_normal((1, 3, 1, 2, 4)), rng.standard_normal((1, 3, 1, 2, 4)))
    for _ in range(10):
        O.decode_step(c, rng.standard_normal((1, 3, 1, 4)), rng.standard_normal((1, 3, 1, 4)),
                      rng.standard_normal((1, 3, 1, 4)))
    O.evict(c, [6, 12, 20])
    assert [c.length(b) for b in range(3)] == [6, 12, 12]
