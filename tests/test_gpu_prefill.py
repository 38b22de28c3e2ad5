"""GPU parity of the prefill path: attention of every prompt position over the positions up to
itself (Eq. 4-5 for t = 1..M) against the float64 oracle, and the cache state it leaves behind."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _qkv(cfg, T, seed):
    r = np.random.default_rng(seed)
    bf = lambda x: W.to_cache_dtype(x, "bf16")
    q = bf(r.standard_normal((cfg.layers, cfg.batch, cfg.q_heads, T, cfg.head_dim)))
    k, v = W.prompt_kv(cfg, seed, n_tokens=T)
    return q, k, v


@pytest.mark.parametrize("T", [1, 17, 64, 65, 200, 512])
@pytest.mark.parametrize("G", [4, 7])
def test_prefill_attention_matches_oracle(T, G):
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=2, kv_heads=2, q_heads=2 * G, prompt=T, budget=max(T, 64),
                                             window=min(8, T), evict_interval=16)
    q, k, v = _qkv(cfg, T, 40 + T + G)
    gpu = H.make_gpu(cfg)
    out = torch.full((cfg.layers, cfg.batch, cfg.q_heads, T, 128), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    gpu.prefill_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out)
    gpu.synchronize()
    gpu.poll_error()
    ref = O.prefill_attention(q, k, v)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert H.rel_err_vectors(got, ref) <= H.TOL_OUT["bf16"]
    # the cache holds the prompt exactly as dynts_prefill would have stored it
    assert gpu.len(0) == T
    for (l, b, h) in [(0, 0, 0), (1, 1, 1)]:
        Kd, Vd, pos, score = gpu.export_slab(l, b, h)
        assert np.array_equal(Kd.float().numpy(), k[l, b, h]) and np.array_equal(Vd.float().numpy(), v[l, b, h])
        assert np.array_equal(pos.numpy(), np.arange(T)) and np.isinf(score.numpy()).all()
    gpu.close()


@pytest.mark.parametrize("T", [130, 320])
def test_prefill_attention_with_several_items_per_cta(T):
    """More (query tile, head) items than the grid has CTAs (two per SM): every CTA walks several
    items back to back -- the loads and the first product of the next item are issued while the
    current one is still in the softmax, half the grid walks its list backwards -- and every row
    still matches the oracle."""
    cfg = W.get_config("c3_qwen7b").scaled(layers=3, batch=4, prompt=T, budget=max(T, 64), window=8, evict_interval=16)
    n_items = -(-T // 128) * cfg.layers * cfg.batch * cfg.q_heads
    assert n_items > 2 * 2 * torch.cuda.get_device_properties(0).multi_processor_count
    q, k, v = _qkv(cfg, T, 90 + T)
    gpu = H.make_gpu(cfg)
    out = torch.full((cfg.layers, cfg.batch, cfg.q_heads, T, 128), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    gpu.prompt_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out)
    gpu.synchronize()
    gpu.poll_error()
    ref = O.prefill_attention(q, k, v)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert H.rel_err_vectors(got, ref) <= H.TOL_OUT["bf16"]
    gpu.close()


@pytest.mark.parametrize("T", [200, 512])
def test_prefill_attention_when_the_row_maximum_keeps_moving(T):
    """Keys whose norm grows along the prompt: the largest logit of a row sits in its latest tiles and
    exceeds the maximum of the tiles before by far more than the slack the kernel allows its
    reference maximum (2^8), so the accumulated output and sum are rescaled again and again."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=2, kv_heads=2, q_heads=8, prompt=T, budget=max(T, 64),
                                             window=8, evict_interval=16)
    q, k, v = _qkv(cfg, T, 300 + T)
    grow = (1.0 + np.arange(T) / 16.0)[None, None, None, :, None]
    k = W.to_cache_dtype(k * grow, "bf16")
    ref = O.prefill_attention(q, k, v)
    # the recipe does what it says: along the last row, a later tile of 64 keys tops everything before it
    # by more than 8 in base-2 units at least once
    qh, kh = q[0, 0, 0].astype(np.float64), k[0, 0, 0].astype(np.float64)
    lg = (qh[T - 1] @ kh.T) / np.sqrt(128.0) * np.log2(np.e)
    tile_max = [lg[j:j + 64].max() for j in range(0, T, 64)]
    assert any(tile_max[j] > max(tile_max[:j]) + 8 for j in range(1, len(tile_max)))
    gpu = H.make_gpu(cfg)
    out = torch.full((cfg.layers, cfg.batch, cfg.q_heads, T, 128), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    gpu.prompt_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out)
    gpu.synchronize()
    gpu.poll_error()
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert H.rel_err_vectors(got, ref) <= H.TOL_OUT["bf16"]
    gpu.close()


def test_decode_after_prefill_attention_continues_the_sequence():
    """The last prefill row and the first decode step are the same operation on consecutive
    tokens: run prefill over T tokens, then decode token T + 1, and compare both with a prefill
    over T + 1 tokens."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, kv_heads=2, q_heads=8, prompt=90, budget=128, window=8,
                                             evict_interval=16)
    T = 90
    q, k, v = _qkv(cfg, T + 1, 77)
    ref = O.prefill_attention(q, k, v)
    gpu = H.make_gpu(cfg)
    out = torch.empty((1, 1, 8, T, 128), dtype=torch.bfloat16, device="cuda:0")
    gpu.prefill_attn(H.dev(q[..., :T, :], cfg), H.dev(k[..., :T, :], cfg), H.dev(v[..., :T, :], cfg), out)
    o1 = torch.empty((1, 1, 8, 128), dtype=torch.bfloat16, device="cuda:0")
    gpu.decode_attn(H.dev(q[..., T, :], cfg), H.dev(k[..., T, :], cfg), H.dev(v[..., T, :], cfg), o1)
    gpu.synchronize()
    assert H.rel_err_vectors(out.float().cpu().numpy(), ref[..., :T, :]) <= H.TOL_OUT["bf16"]
    assert H.rel_err_vectors(o1.float().cpu().numpy(), ref[..., T, :]) <= H.TOL_OUT["bf16"]
    gpu.close()


def test_prefill_attention_rejects_other_shapes():
    import paper_2601_18383_b200 as D
    cfg = W.get_config("c1_tiny_fp32").scaled(prompt=8)
    gpu = H.make_gpu(cfg)
    x = torch.zeros((1, 1, 4, 8, 64), device="cuda:0")
    kv = torch.zeros((1, 1, 1, 8, 64), device="cuda:0")
    with pytest.raises(D.DyntsError) as e:
        gpu.prefill_attn(x, kv, kv, x)
    assert e.value.status == D.DYNTS_ERR_INVALID_ARG and gpu.len(0) == 0
    gpu.close()


def test_prefill_attention_into_a_cache_of_8_bit_rows():
    """The prompt attention reads the caller's bf16 k, v (so its output equals the bf16 cache's bit
    for bit); the fill stores the oracle's E4M3 codes."""
    import paper_2601_18383_b200 as D
    T = 150
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=1, kv_heads=2, q_heads=8, prompt=T, budget=256, window=8,
                                             evict_interval=16)
    q, k, v = _qkv(cfg, T, 91)
    ks, vs = 0.02, 0.07
    a = H.make_gpu(cfg)
    b = D.Cache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window, cfg.evict_interval,
                dtype="bf16_kv8")
    b.set_kv_scale(ks, vs)
    oa = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, T, 128), dtype=torch.bfloat16, device="cuda:0")
    ob = torch.empty_like(oa)
    a.prefill_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), oa)
    b.prefill_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), ob)
    torch.cuda.synchronize()
    assert torch.equal(oa.view(torch.int16), ob.view(torch.int16))
    assert H.rel_err_vectors(ob.float().cpu().numpy().astype(np.float64), O.prefill_attention(q, k, v)) <= H.TOL_OUT["bf16"]
    for (l, h) in [(0, 0), (1, 1)]:
        Kc, Vc, pos, score = b.export_slab(l, 0, h)
        assert np.array_equal(Kc.numpy(), O.fp8_e4m3_encode(k[l, 0, h] / np.float32(ks)))
        assert np.array_equal(Vc.numpy(), O.fp8_e4m3_encode(v[l, 0, h] / np.float32(vs)))
        assert np.array_equal(pos.numpy(), np.arange(T)) and np.isinf(score.numpy()).all()
    a.close(); b.close()


def test_prefill_attention_layer_by_layer_equals_the_all_layers_call():
    """dynts_prefill_attn_layer for layers 0..L-1 leaves the same outputs and the same cache as one
    dynts_prefill_attn over all layers; the lengths appear with the last layer."""
    T = 150
    cfg = W.get_config("c2_llama8b").scaled(layers=3, batch=2, kv_heads=2, q_heads=8, prompt=T, budget=256, window=8,
                                             evict_interval=16)
    q, k, v = _qkv(cfg, T, 93)
    a, b = H.make_gpu(cfg), H.make_gpu(cfg)
    qd, kd, vd = H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg)
    oa = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, T, 128), dtype=torch.bfloat16, device="cuda:0")
    ob = torch.full_like(oa, float("nan"))
    a.prefill_attn(qd, kd, vd, oa, n_pinned=100)
    for l in range(cfg.layers):
        assert b.len(0) == 0
        b.prefill_attn_layer(l, qd[l], kd[l], vd[l], ob[l], n_pinned=100)
    assert b.len(0) == T == b.len(1)
    torch.cuda.synchronize()
    a.poll_error(); b.poll_error()
    assert torch.equal(oa.view(torch.int16), ob.view(torch.int16))
    for sl in [(0, 0, 0), (1, 1, 1), (2, 0, 1)]:
        Ka, Va, pa, sa = a.export_slab(*sl)
        Kb, Vb, pb, sb = b.export_slab(*sl)
        assert torch.equal(H.bits(Ka), H.bits(Kb)) and torch.equal(H.bits(Va), H.bits(Vb))
        assert torch.equal(pa, pb) and torch.equal(H.bits(sa), H.bits(sb))
        assert np.isinf(sa.numpy()[:100]).all() and (sa.numpy()[100:] == 0).all()
    a.close(); b.close()


def test_lengths_are_refreshed_after_graph_replays():
    """A captured decode step advances the lengths on the device only; dynts_cache_refresh_lengths
    brings the host copy up to date, after which a direct eviction sees the rows."""
    from workloads import gen
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=2, prompt=32, budget=128, window=16, evict_interval=32)
    gpu = H.make_gpu(cfg)
    k, v = gen.torch_keys_values(cfg, 94, 100, "cuda:0")
    gpu.prefill(k, v, n_pinned=cfg.prompt)
    q, kn, vn = [x[0] for x in gen.torch_step_ring(cfg, 94, 1, "cuda:0")]
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    gpu.decode_attn(q, kn, vn, out)                    # eager warm-up: 101 rows
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        gpu.set_stream(side)
        with torch.cuda.graph(graph, stream=side):
            gpu.decode_attn(q, kn, vn, out)            # captured, not run: the host copy says 102 afterwards
    gpu.set_stream(torch.cuda.current_stream())
    torch.cuda.synchronize()
    for _ in range(40):
        graph.replay()
    gpu.refresh_lengths()
    assert gpu.len(0) == 141 == gpu.len(1)
    gpu.poll_error()
    H.check_evict_bit_exact(gpu, cfg, 0)
    assert gpu.len(0) == cfg.budget
    gpu.close()
