"""GPU parity of the fused decode step (append + attention + importance accumulation, Eq. 4-6)
against the float64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _lockstep_steps(cfg, steps, seed, cluster, variant, prompt_rows=None, n_pinned=None):
    """Prefill both sides, run `steps` decode steps, compare out / per-step mass / state."""
    gpu = H.make_gpu(cfg, cluster, variant)
    orc = H.make_oracle(cfg)
    T = cfg.prompt if prompt_rows is None else prompt_rows
    pk, pv = W.prompt_kv(cfg, seed, n_tokens=T)
    M = T if n_pinned is None else n_pinned
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg), n_pinned=M)
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64), n_pinned=M)
    stream = W.DecodeStream(cfg, seed)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=H.tdtype(cfg), device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    worst_out, worst_delta = 0.0, 0.0
    for s in range(1, steps + 1):
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta)
        o_ref, d_ref = O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
        gpu.synchronize()
        gpu.poll_error()
        worst_out = max(worst_out, H.rel_err_vectors(out.float().cpu().numpy(), o_ref))
        dh = delta.cpu().numpy()
        for l, b, h, sl in orc.units():
            worst_delta = max(worst_delta, float(np.abs(dh[l, b, h, :sl.n] - d_ref[l][b][h]).max()))
        assert gpu.len(0) == orc.length(0)
    # state after the run: rows, positions, accumulated scores
    worst_score = 0.0
    for l, b, h, sl in orc.units():
        K, V, pos, score = gpu.export_slab(l, b, h)
        assert K.shape[0] == sl.n
        np.testing.assert_array_equal(K.to(torch.float64).numpy(), sl.K[:sl.n])
        np.testing.assert_array_equal(V.to(torch.float64).numpy(), sl.V[:sl.n])
        np.testing.assert_array_equal(pos.numpy(), sl.pos[:sl.n])
        fin = np.isfinite(sl.score[:sl.n])
        assert (np.isinf(score.numpy()) == ~fin).all()
        worst_score = max(worst_score, float(np.abs(score.numpy()[fin] - sl.score[:sl.n][fin]).max()))
    gpu.close()
    return worst_out, worst_delta, worst_score


@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_fp32_generic_small(cluster):
    cfg = W.get_config("c1_tiny_fp32").scaled(layers=2, batch=2, kv_heads=2, q_heads=8, budget=256, evict_interval=64)
    eo, ed, es = _lockstep_steps(cfg, 40, seed=100 + cluster, cluster=cluster, variant=1)
    assert eo <= H.TOL_OUT["fp32"], eo
    assert ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (ed, es)


@pytest.mark.parametrize("variant,cluster", [(1, 1), (1, 4), (2, 1), (2, 2), (2, 4), (2, 8), (3, 1), (3, 2), (0, 0)])
def test_bf16_llama_shape_small(variant, cluster):
    """Llama-like group (G = 4, d = 128), several tiles and a ragged tail, both kernels."""
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=2, prompt=37, budget=512, window=16, evict_interval=64)
    eo, ed, es = _lockstep_steps(cfg, 45, seed=7, cluster=cluster, variant=variant)
    assert eo <= H.TOL_OUT["bf16"], eo
    assert ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (ed, es)


@pytest.mark.parametrize("variant,cluster", [(1, 2), (2, 1), (2, 8), (3, 2), (0, 0)])
def test_bf16_qwen_shape_small(variant, cluster):
    """Qwen-like group (G = 7)."""
    cfg = W.get_config("c3_qwen7b").scaled(layers=1, batch=3, prompt=200, budget=512, window=16, evict_interval=64)
    eo, ed, es = _lockstep_steps(cfg, 33, seed=8, cluster=cluster, variant=variant)
    assert eo <= H.TOL_OUT["bf16"], eo
    assert ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (ed, es)


@pytest.mark.parametrize("G", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("variant", [1, 2, 3])
def test_group_sizes(G, variant):
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, kv_heads=2, q_heads=2 * G, prompt=50, budget=256,
                                             window=8, evict_interval=32)
    eo, ed, es = _lockstep_steps(cfg, 20, seed=20 + G, cluster=2, variant=variant)
    assert eo <= H.TOL_OUT["bf16"] and ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (eo, ed, es)


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_empty_cache_first_token_attends_to_itself(variant):
    """Degenerate case: no prompt.  Step 1 has a single row; alpha = 1, out = v_new, mass = G."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=0, budget=64, window=4, evict_interval=16)
    gpu = H.make_gpu(cfg, 4, variant)   # more CTAs than rows: most ranks own nothing
    stream = W.DecodeStream(cfg, 3)
    q, k, v = stream.step(1)
    out = torch.empty((1, 1, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((1, 1, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta)
    gpu.synchronize()
    o = out.float().cpu().numpy()
    for h in range(cfg.kv_heads):
        for g in range(cfg.group):
            np.testing.assert_array_equal(o[0, 0, h * cfg.group + g], v[0, 0, h])
    assert torch.allclose(delta[0, 0, :, 0].cpu(), torch.full((cfg.kv_heads,), float(cfg.group)), atol=1e-6)
    assert gpu.len(0) == 1
    gpu.close()


def test_head_dim_64_bf16_and_256_fp32_generic():
    for dtype, d in [("bf16", 64), ("fp32", 256), ("fp32", 96)]:
        cfg = W.get_config("c1_tiny_fp32").scaled(head_dim=d, dtype=dtype, kv_heads=2, q_heads=6, prompt=19,
                                                   budget=128, evict_interval=32)
        eo, ed, es = _lockstep_steps(cfg, 12, seed=31, cluster=2, variant=0)
        assert eo <= H.TOL_OUT[dtype] and ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (dtype, d, eo, ed, es)


@pytest.mark.parametrize("variant", [2, 3])
def test_unpinned_prompt_rows_and_partial_pin(variant):
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=1, prompt=40, budget=256, window=8, evict_interval=32)
    eo, ed, es = _lockstep_steps(cfg, 10, seed=41, cluster=2, variant=variant, prompt_rows=90, n_pinned=40)
    assert eo <= H.TOL_OUT["bf16"] and ed <= H.TOL_DELTA and es <= H.TOL_DELTA


@pytest.mark.parametrize("ctas_per_sm", [1, 2])
def test_stream_kernel_many_slabs_per_cta(ctas_per_sm):
    """Streaming kernel with far more slabs than CTAs: a CTA's piece of the chunk list holds
    slabs it finishes alone and, at both ends, slabs it shares with its neighbours; the row
    counts cross a 32-row chunk boundary during the run."""
    cfg = W.get_config("c2_llama8b").scaled(layers=24, batch=5, prompt=57, budget=256, window=8, evict_interval=32)
    eo, ed, es = _lockstep_steps(cfg, 9, seed=51, cluster=ctas_per_sm, variant=3)
    assert eo <= H.TOL_OUT["bf16"] and ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (eo, ed, es)


def test_stream_kernel_one_slab_many_ctas():
    """One KV head, one layer, a long slab: every chunk goes to a different CTA and the last
    arriver combines dozens of partials."""
    cfg = W.get_config("c3_qwen7b").scaled(layers=1, batch=1, kv_heads=1, q_heads=7, prompt=1500, budget=2048,
                                            window=16, evict_interval=64)
    eo, ed, es = _lockstep_steps(cfg, 5, seed=52, cluster=2, variant=3)
    assert eo <= H.TOL_OUT["bf16"] and ed <= H.TOL_DELTA and es <= H.TOL_DELTA, (eo, ed, es)


def test_layer_by_layer_matches_all_layers():
    """dynts_decode_attn_layer over 0..L-1 gives the same state as the all-layer call."""
    cfg = W.get_config("c2_llama8b").scaled(layers=3, batch=2, prompt=64, budget=256, window=8, evict_interval=32)
    a, b = H.make_gpu(cfg), H.make_gpu(cfg)
    pk, pv = W.prompt_kv(cfg, 5)
    for c in (a, b):
        c.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    stream = W.DecodeStream(cfg, 5)
    oa = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    ob = torch.empty_like(oa)
    for s in range(1, 6):
        q, k, v = [H.dev(x, cfg) for x in stream.step(s)]
        a.decode_attn(q, k, v, oa)
        for l in range(cfg.layers):
            b.decode_attn_layer(l, q[l], k[l], v[l], ob[l])
        assert a.len(0) == b.len(0) == cfg.prompt + s
        torch.cuda.synchronize()
        assert torch.equal(oa.view(torch.int16), ob.view(torch.int16))
    import paper_2601_18383_b200 as D
    with pytest.raises(D.DyntsError):
        b.decode_attn_layer(1, q[1], k[1], v[1], ob[1])     # out of order
    sa, sb = a.scores_tensor(), b.scores_tensor()
    assert torch.equal(sa.view(torch.int32), sb.view(torch.int32))
    a.close(); b.close()


def test_host_buffer_entry_point_and_determinism():
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=1, prompt=100, budget=256, window=8, evict_interval=32)
    a, b = H.make_gpu(cfg), H.make_gpu(cfg)
    pk, pv = W.prompt_kv(cfg, 6)
    for c in (a, b):
        c.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    stream = W.DecodeStream(cfg, 6)
    od = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    oh = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16).pin_memory()
    for s in range(1, 5):
        q, k, v = stream.step(s)
        a.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), od)
        # pinned buffers are read by the kernel in place, pageable ones go through staging copies
        qh, kh, vh = [torch.from_numpy(x).to(torch.bfloat16) for x in (q, k, v)]
        if s % 2:
            qh, kh, vh = qh.pin_memory(), kh.pin_memory(), vh.pin_memory()
        b.decode_attn_host(qh, kh, vh, oh)
        torch.cuda.synchronize()
        assert torch.equal(od.cpu().view(torch.int16), oh.view(torch.int16))
    assert torch.equal(a.scores_tensor().view(torch.int32), b.scores_tensor().view(torch.int32))
    a.close(); b.close()


def test_capacity_error_and_inactive_sequences():
    import paper_2601_18383_b200 as D
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=2, prompt=28, budget=32, window=4, evict_interval=2)
    gpu = H.make_gpu(cfg)
    pk, pv = W.prompt_kv(cfg, 9)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    stream = W.DecodeStream(cfg, 9)
    out = torch.zeros((1, 2, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    for s in range(1, 7):
        q, k, v = [H.dev(x, cfg) for x in stream.step(s)]
        gpu.decode_attn(q, k, v, out)
    assert gpu.len(0) == 34 == gpu.capacity
    with pytest.raises(D.DyntsError) as e:
        gpu.decode_attn(q, k, v, out)
    assert e.value.status == D.DYNTS_ERR_CAPACITY and gpu.len(0) == 34
    gpu.evict(0)
    gpu.seq_reset(1)
    out.zero_()
    gpu.decode_attn(q, k, v, out)
    gpu.synchronize()
    assert gpu.len(0) == 33 and gpu.len(1) == 0
    assert out[0, 1].abs().max().item() == 0.0 and out[0, 0].abs().max().item() > 0.0
    gpu.poll_error()
    gpu.close()


def test_batch_larger_than_the_launch_carries_lengths_for():
    """More than 64 sequences: the streaming kernel then reads the lengths from device memory and
    the last block advances them through the ticket, as under stream capture."""
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=70, kv_heads=1, q_heads=4, prompt=20, budget=96, window=8,
                                             evict_interval=16)
    gpu = H.make_gpu(cfg)
    orc = H.make_oracle(cfg)
    pk, pv = W.prompt_kv(cfg, 17)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64))
    stream = W.DecodeStream(cfg, 17)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    for s in range(1, 40):
        q, k, v = stream.step(s)
        gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, delta if s % 2 else None)
        o_ref, d_ref = O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
        assert gpu.len(69) == orc.length(69) == 20 + s
        if s % 5 == 0:
            assert H.rel_err_vectors(out.float().cpu().numpy(), o_ref) <= H.TOL_OUT["bf16"]
    sc = gpu.scores_tensor().cpu().numpy()
    for l, b, h, sl in orc.units():
        fin = np.isfinite(sl.score[:sl.n])
        assert np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max() <= H.TOL_DELTA
        pos = gpu.export_slab(l, b, h)[2].numpy()
        assert np.array_equal(pos, sl.pos[:sl.n])
    gpu.poll_error()
    gpu.close()
