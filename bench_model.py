#!/usr/bin/env python
"""Whole-model decode around the library: a random-init DeepSeek-R1-Distill-Llama-8B-shaped decoder
(32 layers, hidden 4096, 32/8 heads, head_dim 128, MLP 14336, RMSNorm, RoPE theta 500000, vocab
128256, bf16), batch 8, greedy.  Everything but attention runs through PyTorch/cuBLAS; attention,
importance accumulation and eviction run through dynts_decode_attn_layer / dynts_evict.

Two arms are timed in the state a long decode reaches: the budget-limited cache (budget rows per
slab, eviction every E steps) and the full KV cache holding `--context` generated tokens.  The
caches are filled with seeded synthetic K/V rows of that many tokens instead of decoding them one
by one; the timed steps are real decode steps (the model's own q/k/v, RoPE, greedy argmax).

    python bench_model.py [--steps 128] [--context 16384] [--budget 3072]

Prints one JSON line: tokens/s, ms/step and the attention share of each arm, KV bytes in use,
and their ratios.  This is not the benchmark of the hot path (bench.py is); it shows what the hot
path buys inside a model step that also reads 16 GB of weights.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import workloads as W  # noqa: E402
from workloads import gen  # noqa: E402

L, HID, HQ, HKV, D, FF, VOCAB, THETA = 32, 4096, 32, 8, 128, 14336, 128256, 500000.0


class Model:
    def __init__(self, device, seed=0):
        g = torch.Generator(device=device).manual_seed(seed)
        mk = lambda *s: (torch.randn(s, generator=g, device=device) * 0.02).to(torch.bfloat16)
        self.embed = mk(VOCAB, HID)
        self.head = mk(VOCAB, HID)
        self.layers = [dict(wq=mk(HQ * D, HID), wk=mk(HKV * D, HID), wv=mk(HKV * D, HID), wo=mk(HID, HQ * D),
                            wg=mk(FF, HID), wu=mk(FF, HID), wd=mk(HID, FF),
                            n1=torch.ones(HID, device=device, dtype=torch.bfloat16),
                            n2=torch.ones(HID, device=device, dtype=torch.bfloat16)) for _ in range(L)]
        self.nf = torch.ones(HID, device=device, dtype=torch.bfloat16)
        inv = 1.0 / (THETA ** (torch.arange(0, D, 2, device=device, dtype=torch.float32) / D))
        self.inv_freq = inv
        self.weight_bytes = sum(t.numel() * 2 for lay in self.layers for t in lay.values()) + self.head.numel() * 2

    @staticmethod
    def rms(x, w):
        xf = x.float()
        return (xf * torch.rsqrt(xf.pow(2).mean(-1, keepdim=True) + 1e-5)).to(torch.bfloat16) * w

    def rope(self, x, pos):
        """x [Nb, H, D], pos [Nb] -> rotated (half-split convention)."""
        ang = pos.float()[:, None] * self.inv_freq[None, :]                  # [Nb, D/2]
        cos, sin = ang.cos()[:, None, :], ang.sin()[:, None, :]
        xf = x.float()
        a, b = xf[..., : D // 2], xf[..., D // 2:]
        return torch.cat([a * cos - b * sin, a * sin + b * cos], -1).to(torch.bfloat16)

    def step(self, tokens, pos, cache, out_buf, attn_events=None):
        Nb = tokens.shape[0]
        x = self.embed[tokens]
        for l, w in enumerate(self.layers):
            h = self.rms(x, w["n1"])
            q = self.rope((h @ w["wq"].T).view(Nb, HQ, D), pos).contiguous()
            k = self.rope((h @ w["wk"].T).view(Nb, HKV, D), pos).contiguous()
            v = (h @ w["wv"].T).view(Nb, HKV, D).contiguous()
            if attn_events is not None:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
            cache.decode_attn_layer(l, q, k, v, out_buf)
            if attn_events is not None:
                b.record()
                attn_events.append((a, b))
            x = x + out_buf.view(Nb, HQ * D) @ w["wo"].T
            h = self.rms(x, w["n2"])
            x = x + (torch.nn.functional.silu(h @ w["wg"].T) * (h @ w["wu"].T)) @ w["wd"].T
        logits = self.rms(x, self.nf) @ self.head.T
        return logits.argmax(-1)


def make_cache(batch, rows, budget, window, interval, capacity, device, seed):
    import paper_2601_18383_b200 as Dn
    cache = Dn.Cache(L, batch, HQ, HKV, D, budget, window, interval, dtype="bf16", capacity=capacity, device=device)
    cfg = W.get_config("c2_llama8b").scaled(batch=1, density=0.03)
    for b in range(batch):                       # one sequence at a time: bounded temporary memory
        k, v = gen.torch_keys_values(cfg, seed + b, rows, device)
        cache.prefill_seq(b, k[:, 0], v[:, 0], n_pinned=256)
        del k, v
    torch.cuda.empty_cache()
    return cache


def run_arm(model, cache, batch, start_pos, steps, interval, evict, device):
    """Times `steps` decode steps replayed as CUDA graphs (a model step is ~450 small launches, so
    eager PyTorch would measure the host).  Budget arm: one graph = `interval` steps + the eviction,
    which returns the cache to the same lengths, so the graph can be replayed.  Full-KV arm: one
    graph = one step (the lengths live on the device and simply grow)."""
    out_buf = torch.empty((batch, HQ, D), dtype=torch.bfloat16, device=device)
    tokens = torch.arange(batch, device=device) + 1000
    pos = torch.full((batch,), start_pos, device=device, dtype=torch.int64)
    qkv = {}

    def model_step():
        tokens.copy_(model.step(tokens, pos, cache, out_buf))
        pos.add_(1)

    def attn_only_step():                         # the attention calls of one step on fixed q/k/v
        for l in range(L):
            cache.decode_attn_layer(l, qkv["q"], qkv["k"], qkv["v"], out_buf)

    per_graph = interval if evict else 1

    def body(fn):
        for _ in range(per_graph):
            fn()
        if evict:
            cache.evict(0)

    body(model_step)                              # eager warm-up: cuBLAS workspaces, first-call set-up
    g = torch.Generator(device=device).manual_seed(5)
    qkv["q"] = torch.randn((batch, HQ, D), generator=g, device=device).to(torch.bfloat16)
    qkv["k"] = torch.randn((batch, HKV, D), generator=g, device=device).to(torch.bfloat16)
    qkv["v"] = torch.randn((batch, HKV, D), generator=g, device=device).to(torch.bfloat16)
    torch.cuda.synchronize(device)
    side = torch.cuda.Stream(device)
    graphs = {}
    for name, fn in (("model", model_step), ("attention", attn_only_step)):
        gr = torch.cuda.CUDAGraph()
        side.wait_stream(torch.cuda.current_stream(device))
        with torch.cuda.stream(side):
            cache.set_stream(side)
            with torch.cuda.graph(gr, stream=side):
                body(fn)
        graphs[name] = gr
    cache.set_stream(torch.cuda.current_stream(device))
    torch.cuda.synchronize(device)
    reps = max(1, steps // per_graph)
    times = {}
    for name in ("model", "attention"):
        graphs[name].replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            graphs[name].replay()
        b.record()
        torch.cuda.synchronize(device)
        times[name] = a.elapsed_time(b) / (reps * per_graph)
    cache.poll_error()
    rows = cache.len(0) if evict else start_pos + 1 + 2 * (reps + 1)   # the full-KV graphs appended on the device only
    kv_bytes = batch * rows * L * HKV * 2 * D * 2
    return {"tokens_per_s": round(batch / (times["model"] * 1e-3), 1), "ms_per_step": round(times["model"], 3),
            "attention_ms_per_step": round(times["attention"], 3), "kv_bytes_in_use": int(kv_bytes), "rows_per_slab": int(rows),
            "steps_timed": reps * per_graph}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--context", type=int, default=16384, help="tokens generated so far (full-KV arm holds prompt + context)")
    ap.add_argument("--budget", type=int, default=3072)
    ap.add_argument("--window", type=int, default=128)
    ap.add_argument("--interval", type=int, default=64)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("bench_model.py needs a CUDA device")
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    model = Model(device)
    total = 2 * (args.steps + 2) + 8            # the full-KV arm appends in the warm-up, the model graph and the attention graph
    res = {"model": "DeepSeek-R1-Distill-Llama-8B shapes, random init, bf16", "batch": args.batch, "steps": args.steps,
           "weight_bytes_per_step": model.weight_bytes, "data": "synthetic K/V fill + the model's own decode steps"}
    budget_cache = make_cache(args.batch, args.budget, args.budget, args.window, args.interval, 0, device, 100)
    res["budget"] = run_arm(model, budget_cache, args.batch, 256 + args.context, args.steps, args.interval, True, device)
    res["budget"]["budget"] = args.budget
    budget_cache.close()
    torch.cuda.empty_cache()
    full_rows = 256 + args.context
    cap = full_rows + total + 8
    cap = (cap + 31) // 32 * 32
    full_cache = make_cache(args.batch, full_rows, cap, args.window, args.interval, cap, device, 100)
    res["full_kv"] = run_arm(model, full_cache, args.batch, full_rows, args.steps, args.interval, False, device)
    full_cache.close()
    res["speedup"] = round(res["budget"]["tokens_per_s"] / res["full_kv"]["tokens_per_s"], 3)
    res["kv_memory_ratio"] = round(res["full_kv"]["kv_bytes_in_use"] / res["budget"]["kv_bytes_in_use"], 3)
    print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
