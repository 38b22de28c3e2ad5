"""GPU parity of the 8-bit (E4M3) K/V slabs: q, k, v, out stay bf16, the slabs hold codes with one
scale per tensor.  The oracle stores decode(encode(x / scale)) * scale and is otherwise unchanged,
so: the stored codes must equal the oracle's bit for bit (prefill and every appended row, the
saturating ones included), attention outputs and masses must agree within the usual tolerances,
and eviction must move the 128-byte rows bit-exactly."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _make(cfg, ks, vs, variant=0, cluster=0):
    import paper_2601_18383_b200 as D
    gpu = D.Cache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                  cfg.evict_interval, dtype="bf16_kv8")
    gpu.set_launch(cluster, variant)
    gpu.set_kv_scale(ks, vs)
    orc = O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, cfg.capacity,
                        kv_format="e4m3", k_scale=ks, v_scale=vs)
    return gpu, orc


def _codes(x64, scale):
    """Codes of rows the oracle holds (value = decode(code) * scale)."""
    return O.fp8_e4m3_encode((x64 / float(np.float32(scale))).astype(np.float32))


def _check_codes(gpu, orc, ks, vs):
    for l, b, h, sl in orc.units():
        Kc, Vc, pos, _ = gpu.export_slab(l, b, h)
        assert Kc.dtype == torch.uint8 and Kc.shape == (sl.n, orc.head_dim)
        assert np.array_equal(Kc.numpy(), _codes(sl.K[:sl.n], ks)), (l, b, h)
        assert np.array_equal(Vc.numpy(), _codes(sl.V[:sl.n], vs)), (l, b, h)
        assert np.array_equal(pos.numpy(), sl.pos[:sl.n])


@pytest.mark.parametrize("name,ks,vs,variant", [("c2_llama8b", 0.03125, 0.0625, 0), ("c2_llama8b", 0.02, 0.07, 1),
                                                 ("c3_qwen7b", 0.02, 0.07, 0), ("c2_llama8b", 1.0, 1.0, 0)])
def test_trajectory_with_8_bit_slabs(name, ks, vs, variant):
    cfg = W.get_config(name).scaled(layers=2, batch=2, prompt=40, budget=200, window=24, evict_interval=16,
                                    **({"kv_heads": 2, "q_heads": 14} if name == "c3_qwen7b" else {}))
    gpu, orc = _make(cfg, ks, vs, variant)
    pk, pv = W.prompt_kv(cfg, 41)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk, pv)
    _check_codes(gpu, orc, ks, vs)
    stream = W.DecodeStream(cfg, 41)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    worst = dict(out=0.0, delta=0.0, score=0.0)
    events = 0
    for s in range(1, 261):
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta)
        o_ref, d_ref = O.decode_step(orc, q.astype(np.float64), k, v)
        if s % 7 == 0 or s % cfg.evict_interval == 0:
            gpu.synchronize()
            worst["out"] = max(worst["out"], H.rel_err_vectors(out.float().cpu().numpy(), o_ref))
            dh = delta.cpu().numpy()
            for l, b, h, sl in orc.units():
                worst["delta"] = max(worst["delta"], float(np.abs(dh[l, b, h, :sl.n] - d_ref[l][b][h]).max()))
        if s % cfg.evict_interval == 0:
            _check_codes(gpu, orc, ks, vs)                       # every appended row so far
            sc = gpu.scores_tensor().cpu().numpy()
            for l, b, h, sl in orc.units():
                fin = np.isfinite(sl.score[:sl.n])
                worst["score"] = max(worst["score"], float(np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max()))
            n_before = gpu.len(0)
            H.check_evict_bit_exact(gpu, cfg, cfg.budget)       # rows of 128 bytes moved bit for bit
            O.evict(orc, cfg.budget, scores32=lambda l, b, h: sc[l, b, h])
            sc2 = gpu.scores_tensor().cpu().numpy()
            for l, b, h, sl in orc.units():
                assert sl.n == gpu.len(b)
                sl.score[:sl.n] = sc2[l, b, h, :sl.n].astype(np.float64)
            events += int(n_before > cfg.budget)
            _check_codes(gpu, orc, ks, vs)
    gpu.poll_error()
    assert events >= 3
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA and worst["score"] <= H.TOL_DELTA, worst
    gpu.close()


def test_saturation_subnormals_and_the_cost_of_8_bits():
    """Rows far outside the format's range saturate to +-448 x scale, tiny ones land on the subnormal
    grid; and the 8-bit cache's output differs from the bf16 cache's by about the format's error
    (a sanity check that the codes are really used, not a tolerance of the method)."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=64, budget=256, window=16, evict_interval=64)
    gpu, orc = _make(cfg, 1.0, 1.0)
    pk, pv = W.prompt_kv(cfg, 43)
    pk = pk.copy()
    pv = pv.copy()
    pk[..., 3, :] *= 1000.0
    pv[..., 5, :] *= 1e-3
    pk = W.to_cache_dtype(pk, "bf16")
    pv = W.to_cache_dtype(pv, "bf16")
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk, pv)
    _check_codes(gpu, orc, 1.0, 1.0)
    Kc = gpu.export_slab(0, 0, 0)[0].numpy()
    sat = np.abs(pk[0, 0, 0, 3]) >= 448.0
    assert sat.sum() > 32 and ((Kc[3][sat] & 127) == 126).all()       # beyond the largest finite value: saturated
    assert (gpu.export_slab(0, 0, 0)[1].numpy()[5] & 0x78 == 0).all()   # exponent field 0: subnormal or zero
    ref = H.make_gpu(cfg)
    ref.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    stream = W.DecodeStream(cfg, 43)
    q, k, v = stream.step(1)
    out8 = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    out16 = torch.empty_like(out8)
    gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out8)
    ref.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out16)
    o_ref, _ = O.decode_step(orc, q.astype(np.float64), k, v)
    assert H.rel_err_vectors(out8.float().cpu().numpy(), o_ref) <= H.TOL_OUT["bf16"]
    diff = H.rel_err_vectors(out8.float().cpu().numpy(), out16.float().cpu().numpy().astype(np.float64))
    assert 1e-4 < diff
    gpu.close()
    ref.close()


def test_scale_rules():
    import paper_2601_18383_b200 as D
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=8, budget=64, window=8, evict_interval=8)
    gpu, _ = _make(cfg, 0.5, 0.5)
    for bad in ((0.0, 1.0), (1.0, -1.0), (float("inf"), 1.0), (float("nan"), 1.0)):
        with pytest.raises(D.DyntsError):
            gpu.set_kv_scale(*bad)
    pk, pv = W.prompt_kv(cfg, 1)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    with pytest.raises(D.DyntsError):
        gpu.set_kv_scale(1.0, 1.0)                                   # rows are already stored
    gpu.close()
    plain = H.make_gpu(cfg)
    with pytest.raises(D.DyntsError):
        plain.set_kv_scale(1.0, 1.0)                                 # not an 8-bit cache
    plain.close()
    with pytest.raises(D.DyntsError):
        D.Cache(1, 1, 4, 1, 72, 64, 8, 8, dtype="bf16_kv8")          # rows of 72 bytes do not split into 16-byte pieces


def _sampled_full_size(name, seed, rows, ks, vs, n_slabs, steps):
    """Full-size cache in the launch configuration the benchmark times (streaming kernel): sampled
    slabs are exported as codes before each step and the oracle recomputes them one by one."""
    import paper_2601_18383_b200 as D
    from workloads import gen
    cfg = W.get_config(name)
    gpu = D.Cache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                  cfg.evict_interval, dtype="bf16_kv8", seq_budgets=cfg.seq_budgets)
    gpu.set_kv_scale(ks, vs)
    k, v = gen.torch_keys_values(cfg, seed, rows, "cuda:0")
    gpu.prefill(k, v, n_pinned=cfg.prompt)
    del k, v
    r = np.random.default_rng(seed)
    all_ = [(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch) for h in range(cfg.kv_heads)]
    slabs = [all_[i] for i in r.choice(len(all_), size=n_slabs, replace=False)] + [all_[0], all_[-1]]
    ring = gen.torch_step_ring(cfg, seed, steps, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    G = cfg.group
    worst = dict(out=0.0, delta=0.0)
    for s in range(steps):
        pre = {sl: gpu.export_slab(*sl) for sl in slabs}
        q, k, v = ring[0][s], ring[1][s], ring[2][s]
        gpu.decode_attn(q, k, v, out, delta)
        gpu.synchronize()
        gpu.poll_error()
        qh, kh, vh = q.double().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy()
        og, dh = out.float().cpu().numpy(), delta.cpu().numpy()
        for (l, b, h) in slabs:
            Kc, Vc, _, _ = pre[(l, b, h)]
            Kr = np.concatenate([O.fp8_e4m3_decode(Kc.numpy()) * float(np.float32(ks)), O.fp8_e4m3_store(kh[l, b, h], ks)[None]])
            Vr = np.concatenate([O.fp8_e4m3_decode(Vc.numpy()) * float(np.float32(vs)), O.fp8_e4m3_store(vh[l, b, h], vs)[None]])
            alpha = O.attention_weights(qh[l, b, h * G:(h + 1) * G], Kr)
            o_ref = O.attention_output(alpha, Vr)
            worst["out"] = max(worst["out"], H.rel_err_vectors(og[l, b, h * G:(h + 1) * G], o_ref))
            worst["delta"] = max(worst["delta"], float(np.abs(dh[l, b, h, :Kr.shape[0]] - alpha.sum(axis=0)).max()))
            Kn, Vn, _, _ = gpu.export_slab(l, b, h)                      # the appended row's codes
            assert np.array_equal(Kn.numpy()[-1], O.fp8_e4m3_encode(kh[l, b, h] / np.float32(ks)))
            assert np.array_equal(Vn.numpy()[-1], O.fp8_e4m3_encode(vh[l, b, h] / np.float32(vs)))
            assert np.array_equal(Kn.numpy()[:-1], Kc.numpy())
    return gpu, cfg, slabs, worst


def test_config2_full_size_8_bit():
    gpu, cfg, slabs, worst = _sampled_full_size("c2_llama8b", 5100, W.get_config("c2_llama8b").capacity - 3, 0.02, 0.05, 8, 3)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    assert gpu.len(0) == cfg.capacity
    H.check_evict_bit_exact(gpu, cfg, 0, slabs=slabs)
    assert gpu.len(0) == cfg.budget
    gpu.close()


def test_config3_full_size_8_bit():
    gpu, cfg, slabs, worst = _sampled_full_size("c3_qwen7b", 5200, W.get_config("c3_qwen7b").budget + 7, 0.03125, 0.0625, 6, 3)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    gpu.close()
    torch.cuda.empty_cache()


def test_recorded_last_pass_with_8_bit_rows():
    """Equally long slabs that fill the grid, no per-step mass requested: the launch leaves the score
    pass of every CTA's last slab to the next launch.  Scores read back every third step must equal
    the oracle's (which accumulates every step at once)."""
    import paper_2601_18383_b200 as D
    from workloads import gen
    cfg = W.get_config("c2_llama8b").scaled(budget=256, window=16, evict_interval=64, prompt=32)
    ks, vs = 0.03125, 0.0625
    gpu, orc = _make(cfg, ks, vs)
    k, v = gen.torch_keys_values(cfg, 2500, cfg.budget + 3, "cuda:0")
    gpu.prefill(k, v, n_pinned=cfg.prompt)
    O.prefill(orc, k.float().cpu().numpy(), v.float().cpu().numpy(), n_pinned=cfg.prompt)
    ring = gen.torch_step_ring(cfg, 2500, 9, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    launches0 = gpu.launch_count()
    for s in range(9):
        q, kk, vv = ring[0][s], ring[1][s], ring[2][s]
        gpu.decode_attn(q, kk, vv, out)
        o_ref, _ = O.decode_step(orc, q.double().cpu().numpy(), kk.float().cpu().numpy(), vv.float().cpu().numpy())
        if (s + 1) % 3 == 0:
            assert H.rel_err_vectors(out.float().cpu().numpy(), o_ref) <= H.TOL_OUT["bf16"]
            sc = gpu.scores_tensor().cpu().numpy()
            worst = 0.0
            for l, b, h, sl in orc.units():
                fin = np.isfinite(sl.score[:sl.n])
                worst = max(worst, float(np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max()))
            assert worst <= H.TOL_DELTA, (s, worst)
    assert gpu.launch_count() - launches0 == 9 + 3      # three reads applied what was still recorded
    gpu.poll_error()
    gpu.close()
