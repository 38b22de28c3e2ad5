"""Seeded synthetic workloads shaped like budget-limited decode of 7-8B reasoning models.

Only random draws and shapes live here.  Each draw is keyed by (seed, stream id, step), so any
decode step can be regenerated on its own without replaying the ones before it.

Distributions
-------------
``normal``     q, k, v ~ N(0, 1).
``planted``    per (layer, sequence, KV head) a fixed random unit vector u; every query of the
               group is g_q + a*u; a new key is "critical" with probability ``density`` and then
               equals g_k + a*u, otherwise g_k (g ~ N(0, I)).  a^2 = 4*sqrt(head_dim), so the
               scaled logit q.k/sqrt(d) of a critical key has mean +4 and the others mean 0.
``student_t``  k ~ N(0, I) scaled per key by |t| with t ~ Student-t(nu=3) (heavy-tailed norms);
               q, v ~ N(0, 1).

All values are rounded once to the cache dtype (bf16 or fp32) and returned as float32 numpy
arrays that hold exactly representable values of that dtype.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    layers: int
    batch: int
    q_heads: int
    kv_heads: int
    head_dim: int
    prompt: int           # M: pinned question tokens
    decode_steps: int     # T
    budget: int           # B
    window: int           # W
    evict_interval: int   # E
    dtype: str            # "fp32" | "bf16"
    dist: str = "normal"  # "normal" | "planted" | "student_t"
    density: float = 0.0
    seq_budgets: Optional[Tuple[int, ...]] = None   # ragged batches: per-sequence budget
    seq_decode_steps: Optional[Tuple[int, ...]] = None

    @property
    def group(self) -> int:
        return self.q_heads // self.kv_heads

    @property
    def capacity(self) -> int:
        b = max(self.seq_budgets) if self.seq_budgets else self.budget
        return b + self.evict_interval

    def scaled(self, **kw) -> "WorkloadConfig":
        """Same distribution and head shapes with some sizes replaced (shortened parity runs)."""
        return dataclasses.replace(self, **kw)


def _ragged(seed: int, batch: int):
    r = np.random.default_rng([seed, 77])
    budgets = tuple(int(x) for x in r.choice([1024, 2048, 3072], size=batch))
    steps = tuple(int(x) for x in r.integers(4096, 32768 + 1, size=batch))
    return budgets, steps


_RB, _RS = _ragged(4000, 64)

CONFIGS = {
    # tiny fp32 single layer; the CPU oracle replays it in seconds
    "c1_tiny_fp32": WorkloadConfig("c1_tiny_fp32", 1, 1, 4, 1, 64, 32, 512, 128, 16, 32, "fp32", "normal"),
    # Llama-8B-shaped attention stack, batch 1
    "c2_llama8b": WorkloadConfig("c2_llama8b", 32, 1, 32, 8, 128, 256, 16384, 2048, 128, 64, "bf16", "planted", 0.05),
    # Qwen-7B-shaped attention stack, batch 16
    "c3_qwen7b": WorkloadConfig("c3_qwen7b", 28, 16, 28, 4, 128, 512, 32768, 4096, 256, 128, "bf16", "planted", 0.02),
    # ragged throughput batch with Llama-8B attention shapes; prompt 256 and window 128 are chosen
    # here (the workload statement leaves them open)
    "c4_ragged": WorkloadConfig("c4_ragged", 32, 64, 32, 8, 128, 256, 32768, 3072, 128, 64, "bf16", "student_t", 0.0,
                                seq_budgets=_RB, seq_decode_steps=_RS),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name]


def make_rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(s) for s in stream]])


def to_cache_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float values once to the cache dtype; return float32 holding those exact values."""
    x = np.asarray(x, dtype=np.float32)
    if dtype == "fp32":
        return x
    if dtype == "bf16":
        import torch
        return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).to(torch.float32).numpy()
    raise ValueError(dtype)


def _unit_dirs(cfg: WorkloadConfig, seed: int) -> np.ndarray:
    r = make_rng(seed, 1)
    u = r.standard_normal((cfg.layers, cfg.batch, cfg.kv_heads, cfg.head_dim))
    return u / np.linalg.norm(u, axis=-1, keepdims=True)


def _keys(cfg: WorkloadConfig, r: np.random.Generator, u: np.ndarray, n: int) -> np.ndarray:
    """n keys per slab: [L, Nb, Hkv, n, d]."""
    shp = (cfg.layers, cfg.batch, cfg.kv_heads, n, cfg.head_dim)
    k = r.standard_normal(shp)
    if cfg.dist == "planted":
        a = np.sqrt(4.0 * np.sqrt(cfg.head_dim))
        crit = r.random(shp[:-1]) < cfg.density
        k = k + (a * crit)[..., None] * u[:, :, :, None, :]
    elif cfg.dist == "student_t":
        z = r.standard_normal(shp[:-1])
        chi = r.chisquare(3.0, shp[:-1])
        k = k * np.abs(z / np.sqrt(chi / 3.0))[..., None]
    return k


def prompt_kv(cfg: WorkloadConfig, seed: int, n_tokens: Optional[int] = None):
    """Prompt K and V, [L, Nb, Hkv, n_tokens, d] each, in the cache dtype's value set."""
    n = cfg.prompt if n_tokens is None else n_tokens
    u = _unit_dirs(cfg, seed)
    r = make_rng(seed, 2)
    k = _keys(cfg, r, u, n)
    v = r.standard_normal(k.shape)
    return to_cache_dtype(k, cfg.dtype), to_cache_dtype(v, cfg.dtype)


class DecodeStream:
    """Per-step decode inputs: q [L, Nb, Hq, d], k_new and v_new [L, Nb, Hkv, d]."""

    def __init__(self, cfg: WorkloadConfig, seed: int):
        self.cfg = cfg
        self.seed = int(seed)
        self.u = _unit_dirs(cfg, seed)

    def step(self, s: int):
        cfg = self.cfg
        r = make_rng(self.seed, 3, s)
        q = r.standard_normal((cfg.layers, cfg.batch, cfg.kv_heads, cfg.group, cfg.head_dim))
        if cfg.dist == "planted":
            a = np.sqrt(4.0 * np.sqrt(cfg.head_dim))
            q = q + a * self.u[:, :, :, None, :]
        q = q.reshape(cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim)
        k = _keys(cfg, r, self.u, 1)[:, :, :, 0, :]
        v = r.standard_normal(k.shape)
        return (to_cache_dtype(q, cfg.dtype), to_cache_dtype(k, cfg.dtype), to_cache_dtype(v, cfg.dtype))


# ----------------------------------------------------------------------------------------------
# Device-side bulk generation for full-size runs (the same recipes, drawn with a seeded torch
# generator on the GPU so that multi-GB caches need no host round trip).
# ----------------------------------------------------------------------------------------------

def torch_dtype(dtype: str):
    import torch
    return {"bf16": torch.bfloat16, "fp32": torch.float32}[dtype]


def torch_unit_dirs(cfg: WorkloadConfig, seed: int, device):
    import torch
    g = torch.Generator(device=device).manual_seed(int(seed) * 7919 + 1)
    u = torch.randn((cfg.layers, cfg.batch, cfg.kv_heads, cfg.head_dim), generator=g, device=device)
    return u / u.norm(dim=-1, keepdim=True)


def torch_keys_values(cfg: WorkloadConfig, seed: int, n: int, device, u=None):
    """K, V [L, Nb, Hkv, n, d] in the cache dtype, generated on ``device``."""
    import torch
    g = torch.Generator(device=device).manual_seed(int(seed) * 7919 + 2)
    shp = (cfg.layers, cfg.batch, cfg.kv_heads, n, cfg.head_dim)
    dt = torch_dtype(cfg.dtype)
    k = torch.randn(shp, generator=g, device=device, dtype=torch.float32)
    if cfg.dist == "planted":
        if u is None:
            u = torch_unit_dirs(cfg, seed, device)
        a = float(np.sqrt(4.0 * np.sqrt(cfg.head_dim)))
        crit = torch.rand(shp[:-1], generator=g, device=device) < cfg.density
        k += (a * crit.float())[..., None] * u[:, :, :, None, :]
    elif cfg.dist == "student_t":
        z = torch.randn(shp[:-1], generator=g, device=device)
        chi = (torch.randn((3,) + shp[:-1], generator=g, device=device) ** 2).sum(0)
        k *= (z / torch.sqrt(chi / 3.0)).abs()[..., None]
    k = k.to(dt)
    v = torch.randn(shp, generator=g, device=device, dtype=torch.float32).to(dt)
    return k, v


def torch_step_ring(cfg: WorkloadConfig, seed: int, n_steps: int, device, u=None):
    """A ring of decode inputs: q [n, L, Nb, Hq, d], k_new, v_new [n, L, Nb, Hkv, d]."""
    import torch
    g = torch.Generator(device=device).manual_seed(int(seed) * 7919 + 3)
    dt = torch_dtype(cfg.dtype)
    q = torch.randn((n_steps, cfg.layers, cfg.batch, cfg.kv_heads, cfg.group, cfg.head_dim),
                    generator=g, device=device)
    if cfg.dist == "planted":
        if u is None:
            u = torch_unit_dirs(cfg, seed, device)
        a = float(np.sqrt(4.0 * np.sqrt(cfg.head_dim)))
        q += a * u[None, :, :, :, None, :]
    q = q.reshape(n_steps, cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim).to(dt)
    sub = cfg.scaled(layers=cfg.layers * n_steps)
    uu = None if u is None else u.repeat(n_steps, 1, 1, 1)
    if cfg.dist == "planted" and uu is None:
        uu = torch_unit_dirs(cfg, seed, device).repeat(n_steps, 1, 1, 1)
    k, v = torch_keys_values(sub, seed + 1, 1, device, u=uu)
    k = k.reshape(n_steps, cfg.layers, cfg.batch, cfg.kv_heads, cfg.head_dim)
    v = v.reshape(n_steps, cfg.layers, cfg.batch, cfg.kv_heads, cfg.head_dim)
    return q, k, v
