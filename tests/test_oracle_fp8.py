"""Pins of the oracle's 8-bit K/V storage (E4M3: 1 sign, 4 exponent bits with bias 7, 3 mantissa
bits, no infinities, largest finite 448).  The paper has no passage for it; what fixes it is the
format's definition: known code points, the rounding rule checked by brute force on every pair of
neighbours, a library conversion routine, and the error bound of a 3-bit mantissa."""
import numpy as np
import torch

import workloads as W
from oracle import dynts_oracle as O


def test_code_points_of_the_format():
    v = O.fp8_e4m3_values()
    assert v.shape == (127,) and np.all(np.diff(v) > 0)
    assert v[0] == 0.0 and v[1] == 2.0 ** -9 and v[7] == 7 * 2.0 ** -9      # subnormals
    assert v[8] == 2.0 ** -6                                                # smallest normal
    assert v[0x38] == 1.0 and v[0x39] == 1.125 and v[0x40] == 2.0
    assert v[126] == 448.0 and v[125] == 416.0
    assert O.fp8_e4m3_decode(np.array([0x38, 0xB8, 0x7E, 0xFE, 0x80], dtype=np.uint8)).tolist() == [1.0, -1.0, 448.0, -448.0, -0.0]


def test_round_trip_of_every_code():
    codes = np.array([c for c in range(256) if (c & 127) != 127], dtype=np.uint8)
    assert np.array_equal(O.fp8_e4m3_encode(O.fp8_e4m3_decode(codes)), codes)


def test_nearest_with_ties_to_even_by_brute_force():
    v = O.fp8_e4m3_values()
    for i in range(126):
        lo, hi = v[i], v[i + 1]
        mid = 0.5 * (lo + hi)                                   # exact in float32 (one more mantissa bit)
        assert np.float32(mid) == mid
        even = i if i % 2 == 0 else i + 1
        assert O.fp8_e4m3_encode(np.array([mid]))[0] == even, i
        below, above = np.nextafter(np.float32(mid), np.float32(0)), np.nextafter(np.float32(mid), np.float32(1e9))
        assert O.fp8_e4m3_encode(np.array([below]))[0] == i
        assert O.fp8_e4m3_encode(np.array([above]))[0] == i + 1
        assert O.fp8_e4m3_encode(np.array([-mid]))[0] == even + 128


def test_saturation_and_error_bound():
    big = np.array([448.0, 449.0, 464.0, 480.0, 1e30, -1e30], dtype=np.float32)
    assert O.fp8_e4m3_decode(O.fp8_e4m3_encode(big)).tolist() == [448.0, 448.0, 448.0, 448.0, 448.0, -448.0]
    x = (np.random.default_rng(3).standard_normal(100000) * 20).astype(np.float32)
    y = O.fp8_e4m3_decode(O.fp8_e4m3_encode(x))
    normal = (np.abs(x) >= 2.0 ** -6) & (np.abs(x) <= 448)
    assert np.all(np.abs(y - x)[normal] <= np.abs(x)[normal] * 2.0 ** -4)       # half an ulp of 3 mantissa bits
    assert np.all(np.abs(y - x)[~normal & (np.abs(x) < 2.0 ** -6)] <= 2.0 ** -10)  # half a subnormal step


def test_against_a_library_conversion():
    r = np.random.default_rng(4)
    x = np.concatenate([(r.standard_normal(300000) * s).astype(np.float32) for s in (0.01, 1.0, 40.0, 300.0)])
    ref = torch.from_numpy(x).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(O.fp8_e4m3_encode(x), ref)


def test_store_divides_in_float32_and_scales_back():
    x = np.array([3.3, -0.7, 100.0, 5000.0], dtype=np.float32)
    s = 8.0
    assert O.fp8_e4m3_store(x, s).tolist() == [3.25, -0.6875, 96.0, 3584.0]     # x/8 -> 0.40625, -0.0859375, 12, 448


def test_cache_with_8_bit_rows_is_the_plain_cache_on_stored_values():
    cfg = W.get_config("c1_tiny_fp32").scaled(layers=1, batch=1, prompt=5, budget=40, window=4, evict_interval=8)
    ks, vs = 0.5, 0.25
    a = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, cfg.capacity,
                      kv_format="e4m3", k_scale=ks, v_scale=vs)
    b = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, cfg.capacity)
    pk, pv = W.prompt_kv(cfg, 2)
    O.prefill(a, pk, pv)
    O.prefill(b, O.fp8_e4m3_store(pk, ks), O.fp8_e4m3_store(pv, vs))
    stream = W.DecodeStream(cfg, 2)
    for s in range(1, 12):
        q, k, v = stream.step(s)
        oa, da = O.decode_step(a, q.astype(np.float64), k, v)
        ob, db = O.decode_step(b, q.astype(np.float64), O.fp8_e4m3_store(k, ks), O.fp8_e4m3_store(v, vs))
        assert np.array_equal(oa, ob)
        if s % 8 == 0:
            O.evict(a, cfg.budget // 2)
            O.evict(b, cfg.budget // 2)
    sa, sb = a.slab(0, 0, 0), b.slab(0, 0, 0)
    assert sa.n == sb.n and np.array_equal(sa.K[:sa.n], sb.K[:sb.n]) and np.array_equal(sa.score[:sa.n], sb.score[:sb.n])
    # the stored rows really are on the 8-bit grid, and they differ from the inputs
    codes = O.fp8_e4m3_encode((sa.K[:sa.n] / ks).astype(np.float32))
    assert np.array_equal(O.fp8_e4m3_decode(codes) * ks, sa.K[:sa.n])
    assert not np.array_equal(sa.K[:5], pk[0, 0, 0, :5].astype(np.float64))
