"""dynts_evict_noalloc: the eviction for callers that must not allocate device memory.

A serving loop that froze its allocator after start-up, or code running inside a memory pool's
critical section, cannot create a cache object (whose storage holds the gather list between the
selection and compaction kernels).  This entry point keeps that list in an array built into the
library instead.  The test drives it through the C ABI on caller-owned slabs and requires the
result to equal the cache object's eviction bit for bit (indices, K, V, pos, score), twice in a
row so that contents left behind by the first call cannot leak into the second.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _reference_and_inputs(cfg, rows, seed):
    """Fill a cache, give it scores, snapshot its slabs into plain tensors, evict the cache."""
    gpu = H.make_gpu(cfg)
    k, v = W.prompt_kv(cfg, seed, n_tokens=rows)
    gpu.prefill(H.dev(k, cfg), H.dev(v, cfg), n_pinned=cfg.prompt)
    sc = gpu.scores_tensor()
    g = torch.Generator(device="cuda").manual_seed(seed)
    vals = torch.randint(0, 50, sc[..., cfg.prompt:rows].shape, generator=g, device="cuda").float() / 7.0   # ties
    sc[..., cfg.prompt:rows] = vals
    torch.cuda.synchronize()
    slabs = cfg.layers * cfg.batch * cfg.kv_heads
    cap, d = gpu.capacity, cfg.head_dim
    dt = H.tdtype(cfg)
    K = torch.zeros((slabs, cap, d), dtype=dt, device="cuda")
    V = torch.zeros((slabs, cap, d), dtype=dt, device="cuda")
    pos = torch.zeros((slabs, cap), dtype=torch.int32, device="cuda")
    score = torch.zeros((slabs, cap), dtype=torch.float32, device="cuda")
    i = 0
    for l in range(cfg.layers):
        for b in range(cfg.batch):
            for h in range(cfg.kv_heads):
                Ks, Vs, ps, ss = gpu.export_slab(l, b, h)
                K[i, :rows], V[i, :rows], pos[i, :rows], score[i, :rows] = Ks.cuda(), Vs.cuda(), ps.cuda(), ss.cuda()
                i += 1
    gpu.evict(cfg.budget)
    ref = [gpu.export_slab(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch) for h in range(cfg.kv_heads)]
    gpu.close()
    return (K, V, pos, score), ref, cap


def _check(cfg, rows, seed):
    import paper_2601_18383_b200 as D
    (K, V, pos, score), ref, cap = _reference_and_inputs(cfg, rows, seed)
    slabs = K.shape[0]
    D.dynts_evict_noalloc(K, V, pos, score, slabs, cfg.head_dim, D.DYNTS_BF16 if cfg.dtype == "bf16" else D.DYNTS_FP32,
                          cap, rows, cfg.prompt, cfg.window, cfg.budget,
                          torch.cuda.current_stream().cuda_stream)
    D.dynts_evict_noalloc_status(torch.cuda.current_stream().cuda_stream)   # waits; raises if a device-side check fired
    n = min(rows, cfg.budget)
    for i, (Kr, Vr, pr, sr) in enumerate(ref):
        assert Kr.shape[0] == n
        assert torch.equal(pos[i, :n].cpu(), pr)
        assert torch.equal(H.bits(score[i, :n].cpu()), H.bits(sr))
        assert torch.equal(H.bits(K[i, :n].cpu()), H.bits(Kr))
        assert torch.equal(H.bits(V[i, :n].cpu()), H.bits(Vr))


def test_noalloc_matches_cache_eviction_twice_in_a_row():
    big = W.get_config("c2_llama8b").scaled(layers=2, batch=2, prompt=40, budget=900, window=64, evict_interval=300)
    small = W.get_config("c1_tiny_fp32").scaled(layers=1, batch=3, kv_heads=2, q_heads=8, prompt=8, budget=100, window=16,
                                                evict_interval=60)
    _check(big, 1187, seed=11)        # first call: leaves a long gather list behind
    _check(small, 151, seed=12)       # second call: other dtype, fewer and shorter slabs
    _check(big, 1200, seed=13)        # and a third with the first shape again


def test_noalloc_rejects_oversize_and_bad_arguments():
    import paper_2601_18383_b200 as D
    K = torch.zeros((1, 16, 128), dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros((1, 16), dtype=torch.int32, device="cuda")
    sc = torch.zeros((1, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(D.DyntsError) as e:      # 2048 slabs x 2112 rows do not fit the built-in scratch
        D.dynts_evict_noalloc(K, K, pos, sc, 2048, 128, D.DYNTS_BF16, 2112, 2112, 256, 128, 2048, None)
    assert e.value.status == D.DYNTS_ERR_CAPACITY and "scratch" in str(e.value)
    with pytest.raises(D.DyntsError) as e:
        D.dynts_evict_noalloc(K, K, pos, sc, 1, 128, D.DYNTS_BF16, 16, 16, 8, 8, 12, None)
    assert e.value.status == D.DYNTS_ERR_BUDGET
    with pytest.raises(D.DyntsError):
        D.dynts_evict_noalloc(None, K, pos, sc, 1, 128, D.DYNTS_BF16, 16, 16, 0, 0, 8, None)
    D.dynts_evict_noalloc(K, K, pos, sc, 1, 128, D.DYNTS_BF16, 16, 10, 0, 0, 12, None)   # n <= target: no-op


def test_noalloc_moves_rows_of_8_bit_codes():
    """Slabs of E4M3 codes (128-byte rows): the selection is the oracle's, the rows move bit for bit."""
    import paper_2601_18383_b200 as D
    from oracle import dynts_oracle as O
    slabs, cap, d, rows, pinned, window, target = 5, 400, 128, 389, 24, 32, 200
    g = torch.Generator(device="cuda").manual_seed(21)
    K = torch.randint(0, 256, (slabs, cap, d), generator=g, device="cuda", dtype=torch.uint8)
    V = torch.randint(0, 256, (slabs, cap, d), generator=g, device="cuda", dtype=torch.uint8)
    pos = torch.arange(cap, dtype=torch.int32, device="cuda").repeat(slabs, 1).contiguous()
    score = (torch.randint(0, 40, (slabs, cap), generator=g, device="cuda").float() / 3.0).contiguous()   # ties
    score[:, :pinned] = float("inf")
    K0, V0, s0 = K.cpu(), V.cpu(), score.cpu()
    D.dynts_evict_noalloc(K, V, pos, score, slabs, d, D.DYNTS_BF16_KV8, cap, rows, pinned, window, target,
                          torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for i in range(slabs):
        kept = torch.from_numpy(O.select_keep(s0[i, :rows].numpy(), rows, pinned, window, target))
        assert len(kept) == target
        assert torch.equal(pos[i, :target].cpu(), kept.to(torch.int32))
        assert torch.equal(K[i, :target].cpu(), K0[i][kept]) and torch.equal(V[i, :target].cpu(), V0[i][kept])
        assert torch.equal(H.bits(score[i, :target].cpu()), H.bits(s0[i][kept]))
