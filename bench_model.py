#!/usr/bin/env python
"""Whole-model decode around the library: a random-init DeepSeek-R1-Distill-Llama-8B-shaped decoder
(32 layers, hidden 4096, 32/8 heads, head_dim 128, MLP 14336, RMSNorm, RoPE theta 500000, vocab
128256, bf16), batch 8, greedy.  Everything but attention runs through PyTorch/cuBLAS; attention,
importance accumulation and eviction run through dynts_decode_attn_layer / dynts_evict.

Default mode, the whole trajectory: a 256-token prompt (seeded random token ids) goes through the
model with dynts_prefill_attn_layer, then `--tokens` tokens (4096; 16384 is the workload as stated)
are decoded greedily, one CUDA-graph replay per step, in two arms: the budget-limited cache
(budget 3072, an eviction whenever the length has grown by the interval of 64 beyond it) and a
full KV cache.  Per arm: tokens/s over the run and over the last 512 steps, the attention time per
step at the end, the length / time sawtooth per 64-step chunk (beside Section 5's closed form for
the length), peak KV rows and bytes; across arms: speed-up, KV memory ratio and Appendix A's
attention-flop ratio.

    python bench_model.py [--tokens 4096] [--budget 3072] [--out model_loop.json]

`--late-state` instead times 128 steps in the state a 16384-token decode reaches, the caches
filled with seeded synthetic K/V rows (no trajectory, no evictions falling due).

Prints one JSON line.  This is not the benchmark of the hot path (bench.py is); it shows what the
hot path buys inside a model step that also reads 16 GB of weights.
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

    def rope_seq(self, x):
        """x [Nb, T, H, D] at positions 0..T-1 -> rotated."""
        T = x.shape[1]
        ang = torch.arange(T, device=x.device, dtype=torch.float32)[:, None] * self.inv_freq[None, :]   # [T, D/2]
        cos, sin = ang.cos()[None, :, None, :], ang.sin()[None, :, None, :]
        xf = x.float()
        a, b = xf[..., : D // 2], xf[..., D // 2:]
        return torch.cat([a * cos - b * sin, a * sin + b * cos], -1).to(torch.bfloat16)

    def prefill(self, prompt, cache):
        """The prompt through all layers (attention and the fill of the question window by
        dynts_prefill_attn_layer); returns the first generated token of every sequence."""
        Nb, T = prompt.shape
        x = self.embed[prompt]                                               # [Nb, T, HID]
        out = torch.empty((Nb, HQ, T, D), dtype=torch.bfloat16, device=x.device)
        for l, w in enumerate(self.layers):
            h = self.rms(x, w["n1"])
            q = self.rope_seq((h @ w["wq"].T).view(Nb, T, HQ, D)).permute(0, 2, 1, 3).contiguous()
            k = self.rope_seq((h @ w["wk"].T).view(Nb, T, HKV, D)).permute(0, 2, 1, 3).contiguous()
            v = (h @ w["wv"].T).view(Nb, T, HKV, D).permute(0, 2, 1, 3).contiguous()
            cache.prefill_attn_layer(l, q, k, v, out, n_pinned=T)
            x = x + out.permute(0, 2, 1, 3).reshape(Nb, T, HQ * D) @ w["wo"].T
            h = self.rms(x, w["n2"])
            x = x + (torch.nn.functional.silu(h @ w["wg"].T) * (h @ w["wu"].T)) @ w["wd"].T
        logits = self.rms(x[:, -1], self.nf) @ self.head.T
        return logits.argmax(-1)

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


def run_trajectory(model, args, limited, device):
    """One arm of the whole trajectory: prompt through the model, then args.tokens greedy steps."""
    import paper_2601_18383_b200 as Dn
    batch, M, E, B = args.batch, args.prompt, args.interval, args.budget
    if limited:
        budget, cap = B, B + E
    else:
        cap = (M + args.tokens + 48 + 31) // 32 * 32
        budget = cap
    cache = Dn.Cache(L, batch, HQ, HKV, D, budget, args.window, E, dtype="bf16", capacity=cap, device=device)
    g = torch.Generator(device=device).manual_seed(11)
    prompt = torch.randint(0, VOCAB, (batch, M), generator=g, device=device)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    first = model.prefill(prompt, cache)
    t1.record()
    torch.cuda.synchronize(device)
    prefill_ms = t0.elapsed_time(t1)
    assert cache.len(0) == M
    out_buf = torch.empty((batch, HQ, D), dtype=torch.bfloat16, device=device)
    tokens = first.clone()
    pos = torch.full((batch,), M, device=device, dtype=torch.int64)

    def model_step():
        tokens.copy_(model.step(tokens, pos, cache, out_buf))
        pos.add_(1)

    model_step()                                   # eager: first-call set-up; the first decoded token
    torch.cuda.synchronize(device)
    side = torch.cuda.Stream(device)
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream(device))
    with torch.cuda.stream(side):
        cache.set_stream(side)
        with torch.cuda.graph(graph, stream=side):
            model_step()                           # captured, not run
    cache.set_stream(torch.cuda.current_stream(device))
    cache.refresh_lengths()                        # the capture advanced the host copy only
    done = 1
    chunks = []                                    # (steps done, rows before eviction, rows after, ms per step)
    peak_rows = cache.len(0)
    evict_ms_total = 0.0
    ev = lambda: torch.cuda.Event(enable_timing=True)
    while done < args.tokens:
        n = min(E - done % E, args.tokens - done)
        a, b = ev(), ev()
        a.record()
        for _ in range(n):
            graph.replay()
        b.record()
        cache.refresh_lengths()                    # synchronises
        done += n
        rows = cache.len(0)
        peak_rows = max(peak_rows, rows)
        ev_ms = 0.0
        if limited and rows > B:
            c0, c1 = ev(), ev()
            c0.record()
            cache.evict(0)
            c1.record()
            torch.cuda.synchronize(device)
            ev_ms = c0.elapsed_time(c1)
        evict_ms_total += ev_ms
        chunks.append((done, rows, cache.len(0), a.elapsed_time(b) / n))
        cache.poll_error()
    # Section 5's closed form with the trigger at B + E and E rows leaving per event
    ok = all(after == ((M + d if M + d <= B else B) if limited else M + d) for d, _, after, _ in chunks if d % E == 0)
    total_ms = evict_ms_total + sum(ms * (d - (chunks[i - 1][0] if i else 1)) for i, (d, _, _, ms) in enumerate(chunks))
    tail = [(d, ms) for d, _, _, ms in chunks if d > args.tokens - 512]
    tail_ms = sum(ms for _, ms in tail) / max(1, len(tail))
    # attention alone at the end of the run: the 32 layer calls of a step on fixed q, k, v
    gq = torch.Generator(device=device).manual_seed(5)
    aq = torch.randn((batch, HQ, D), generator=gq, device=device).to(torch.bfloat16)
    ak = torch.randn((batch, HKV, D), generator=gq, device=device).to(torch.bfloat16)
    av = torch.randn((batch, HKV, D), generator=gq, device=device).to(torch.bfloat16)
    reps = 8
    a, b = ev(), ev()
    for l in range(L):
        cache.decode_attn_layer(l, aq, ak, av, out_buf)
    a.record()
    for _ in range(reps):
        for l in range(L):
            cache.decode_attn_layer(l, aq, ak, av, out_buf)
    b.record()
    torch.cuda.synchronize(device)
    attn_ms = a.elapsed_time(b) / reps
    cache.poll_error()
    kv_row_bytes = L * HKV * 2 * D * 2
    res = {"tokens": args.tokens, "prefill_ms": round(prefill_ms, 2),
           "tokens_per_s": round(batch * (args.tokens - 1) / (total_ms * 1e-3), 1),
           "tokens_per_s_last_512": round(batch / (tail_ms * 1e-3), 1),
           "ms_per_step_first_chunks": [round(ms, 3) for _, _, _, ms in chunks[:3]],
           "ms_per_step_last_chunks": [round(ms, 3) for _, _, _, ms in chunks[-3:]],
           "attention_ms_per_step_at_end": round(attn_ms, 3), "attention_us_per_layer_call_at_end": round(attn_ms * 1e3 / L, 2),
           "rows_at_end": chunks[-1][2], "peak_rows_per_slab": int(peak_rows), "peak_kv_bytes": int(batch * peak_rows * kv_row_bytes),
           "allocated_cache_bytes": int(cache.nbytes), "lengths_match_closed_form": bool(ok),
           "evictions": sum(1 for _, r, a2, _ in chunks if a2 < r), "eviction_ms_total": round(evict_ms_total, 3)}
    series = [{"step": d, "rows": r, "rows_after_eviction": a2, "ms_per_step": round(ms, 4)} for d, r, a2, ms in chunks]
    cache.close()
    torch.cuda.empty_cache()
    return res, series


def main_trajectory(args, device):
    model = Model(device)
    res = {"model": "DeepSeek-R1-Distill-Llama-8B shapes, random init, bf16", "batch": args.batch, "prompt": args.prompt,
           "tokens": args.tokens, "budget": args.budget, "window": args.window, "evict_interval": args.interval,
           "weight_bytes_per_step": model.weight_bytes, "data": "seeded random prompt ids; the model's own greedy tokens"}
    res["budget_arm"], s_b = run_trajectory(model, args, True, device)
    res["full_kv_arm"], s_f = run_trajectory(model, args, False, device)
    res["speedup"] = round(res["budget_arm"]["tokens_per_s"] / res["full_kv_arm"]["tokens_per_s"], 3)
    res["speedup_last_512"] = round(res["budget_arm"]["tokens_per_s_last_512"] / res["full_kv_arm"]["tokens_per_s_last_512"], 3)
    res["kv_memory_ratio"] = round(res["full_kv_arm"]["peak_kv_bytes"] / res["budget_arm"]["peak_kv_bytes"], 3)
    # Appendix A: attention flops per step are proportional to the rows attended; Section 5: S_i = M + i - n_i K
    M, B, E = args.prompt, args.budget, args.interval
    s_full = sum(M + i for i in range(1, args.tokens + 1))
    s_lim = sum((M + i) if M + i <= B + E else B + ((M + i - B - 1) % E) + 1 for i in range(1, args.tokens + 1))
    res["attention_flop_ratio_appendix_a"] = round(s_full / s_lim, 3)
    res["attention_time_ratio_at_end"] = round(res["full_kv_arm"]["attention_ms_per_step_at_end"] / res["budget_arm"]["attention_ms_per_step_at_end"], 3)
    if args.out:
        os.makedirs(os.path.dirname(os.path.abspath(args.out)), exist_ok=True)
        with open(args.out, "w") as f:
            json.dump({"summary": res, "budget_arm_series": s_b, "full_kv_arm_series": s_f}, f)
    print(json.dumps(res), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=4096, help="tokens decoded per sequence in the default (trajectory) mode")
    ap.add_argument("--prompt", type=int, default=256)
    ap.add_argument("--out", default="", help="also write the summary and the per-chunk series to this JSON file")
    ap.add_argument("--late-state", action="store_true", help="time --steps steps in the late-decode state on synthetic K/V fills")
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
    if not args.late_state:
        return main_trajectory(args, device)
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
