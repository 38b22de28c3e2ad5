"""Shared helpers of the GPU parity tests: run the CUDA library and the float64 oracle side by
side on the same seeded inputs and compare them."""
import numpy as np
import torch

import workloads as W
from oracle import dynts_oracle as O

TOL_OUT = {"bf16": 1e-2, "fp32": 2e-5}   # max relative error of an output vector (inf-norm)
TOL_DELTA = 1e-4                          # absolute error of a row's attention mass / score


def tdtype(cfg):
    return {"bf16": torch.bfloat16, "fp32": torch.float32}[cfg.dtype]


def dev(x32, cfg, device="cuda:0"):
    """float32 numpy holding cache-dtype values -> device tensor of the cache dtype (exact)."""
    return torch.from_numpy(np.ascontiguousarray(x32)).to(tdtype(cfg)).to(device).contiguous()


def make_gpu(cfg, cluster=0, variant=0, seq_budgets=None, capacity=0):
    import paper_2601_18383_b200 as D
    c = D.Cache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                cfg.evict_interval, dtype=cfg.dtype, seq_budgets=seq_budgets or cfg.seq_budgets, capacity=capacity)
    c.set_launch(cluster, variant)
    return c


def make_oracle(cfg, capacity=None):
    return O.OracleCache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window,
                         capacity or cfg.capacity)


def oracle_from_gpu(gpu, cfg, slabs=None, pinned=None):
    """Build oracle state (float64) from the device cache; only `slabs` [(l, b, h)] if given."""
    orc = make_oracle(cfg, gpu.capacity)
    todo = slabs if slabs is not None else [(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch)
                                            for h in range(cfg.kv_heads)]
    for (l, b, h) in todo:
        K, V, pos, score = gpu.export_slab(l, b, h)
        s = orc.slab(l, b, h)
        n = K.shape[0]
        s.K[:n] = K.to(torch.float64).numpy()
        s.V[:n] = V.to(torch.float64).numpy()
        s.pos[:n] = pos.numpy()
        s.score[:n] = score.to(torch.float64).numpy()
        s.n = n
        orc.next_pos[b] = int(pos[-1]) + 1 if n else 0
    for b in range(cfg.batch):
        orc.n_pinned[b] = cfg.prompt if pinned is None else pinned[b]
    return orc


def rel_err_vectors(out_gpu, out_ref):
    """max over output vectors of ||o - o_ref||_inf / ||o_ref||_inf."""
    g = np.asarray(out_gpu, dtype=np.float64)
    r = np.asarray(out_ref, dtype=np.float64)
    num = np.abs(g - r).max(axis=-1)
    den = np.abs(r).max(axis=-1)
    den = np.where(den == 0, 1.0, den)
    return float((num / den).max())


def export_all(gpu, cfg):
    return {(l, b, h): gpu.export_slab(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch)
            for h in range(cfg.kv_heads)}


def bits(t):
    """Raw bit view for exact comparisons."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16)
    if t.dtype == torch.float32:
        return t.view(torch.int32)
    return t


def check_evict_bit_exact(gpu, cfg, target, pinned=None, slabs=None):
    """Export, evict on the device, and require the result to equal the oracle's selection applied
    to the device's own pre-eviction state, bit for bit.  Returns kept indices per slab."""
    todo = slabs if slabs is not None else [(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch)
                                            for h in range(cfg.kv_heads)]
    pre = {s: gpu.export_slab(*s) for s in todo}
    if isinstance(target, (list, tuple)):
        gpu.evict_ex(list(target))
    else:
        gpu.evict(target)
    gpu.synchronize()
    gpu.poll_error()
    kept_all = {}
    for s in todo:
        K0, V0, p0, s0 = pre[s]
        n = K0.shape[0]
        b = s[1]
        tgt = target[b] if isinstance(target, (list, tuple)) else (target if target > 0 else
              (cfg.seq_budgets[b] if cfg.seq_budgets else cfg.budget))
        M = cfg.prompt if pinned is None else pinned[b]
        kept = O.select_keep(s0.numpy(), n, M, cfg.window, tgt)
        K1, V1, p1, s1 = gpu.export_slab(*s)
        idx = torch.from_numpy(kept)
        assert K1.shape[0] == len(kept), (s, K1.shape[0], len(kept))
        assert torch.equal(p1, p0[idx]), f"pos mismatch in slab {s}"
        assert torch.equal(bits(s1), bits(s0[idx])), f"score mismatch in slab {s}"
        assert torch.equal(bits(K1), bits(K0[idx])), f"K mismatch in slab {s}"
        assert torch.equal(bits(V1), bits(V0[idx])), f"V mismatch in slab {s}"
        kept_all[s] = kept
    return kept_all
