#!/usr/bin/env python
"""The paper's trigger (select when the row count reaches B, keep ratio x W_s; Section 4.2) run as
a long decode on the device, with the analytic curves printed beside the measured ones:

  * cache length per step -- measured (the library's length) against Section 5's closed form
    S_i = M + i - n_i K (a sawtooth between B - K and B);
  * attention work -- Appendix A's 4 L d S_i flops per step summed over the run against the full
    cache's 4 L d (M + i), the predictor's 6 d^2 + d per step, and Eq. 9's net saving at the end;
  * decode time per step -- measured with CUDA events, as a function of the row count, against
    the time the same kernel needs at the full cache's length (a linear fit of the measured
    points extrapolated; the decode step is HBM-bound, so time is linear in rows).

    python bench_schedule.py [--preset dynts] [--workload c2_llama8b] [--steps 4096] [--ratio 0.3]

Prints one JSON line.  Inputs are seeded synthetic tensors shaped like the workload; the predictor
scores are seeded random numbers (the selection does not care where a score comes from).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import workloads as W  # noqa: E402
from workloads import gen  # noqa: E402


def main():
    from paper_2601_18383_b200 import presets as P
    ap = argparse.ArgumentParser()
    ap.add_argument("--preset", default="dynts", choices=P.NAMES)
    ap.add_argument("--workload", default="c2_llama8b", choices=sorted(W.CONFIGS))
    ap.add_argument("--steps", type=int, default=4096)
    ap.add_argument("--ratio", type=float, default=0.3)
    ap.add_argument("--budget", type=int, default=0, help="B (default: the workload's budget)")
    ap.add_argument("--window", type=int, default=-1, help="W_l (default: the workload's window)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("bench_schedule.py needs a CUDA device")
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    cfg = W.get_config(args.workload)
    B = args.budget or cfg.budget
    WL = cfg.window if args.window < 0 else args.window
    M = cfg.prompt
    preset = P.make(args.preset, B, WL, args.ratio, M)
    cfg = cfg.scaled(budget=B, window=preset.window, evict_interval=1, seq_budgets=None)
    run = P.PresetRun(preset, cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, dtype=cfg.dtype, device=device)
    pk, pv = gen.torch_keys_values(cfg, 11, M, device)
    run.prefill(pk, pv)
    ring = 16
    q, k, v = gen.torch_step_ring(cfg, 13, ring, device)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=q.dtype, device=device)
    g = torch.Generator(device=device).manual_seed(17)
    pred = torch.randn((args.steps, cfg.batch), generator=g, device=device)
    rnd = torch.rand((args.steps, cfg.batch), generator=g, device=device)
    st = torch.cuda.current_stream(device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    measured, rows_at_step = [], []
    for s in range(args.steps):
        j = s % ring
        rows_at_step.append(run.cache.len(0) + 1)          # rows the decode kernel of this step reads
        ev[s][0].record(st)
        run.cache.decode_attn(q[j], k[j], v[j], out)
        ev[s][1].record(st)
        sc = preset.step_scores(pred[s], rnd[s])
        if sc is not None:
            run.cache.append_scores(sc)
        before = run.cache.len(0)
        run.cache.evict_at_budget(B, preset.ratio)
        run.events += int(run.cache.len(0) < before)
        measured.append(run.cache.len(0))
    torch.cuda.synchronize(device)
    run.cache.poll_error()
    us = [a.elapsed_time(b) * 1e3 for a, b in ev]
    closed = preset.lengths(M, args.steps)
    K = preset.evicted_per_event()
    n_closed, prev = 0, M
    for c in closed:
        n_closed += int(c < prev + 1)
        prev = c

    # decode time against rows: least squares over the steady part of the run (skip the first steps)
    skip = min(64, args.steps // 4)
    xs = torch.tensor(rows_at_step[skip:], dtype=torch.float64)
    ys = torch.tensor(us[skip:], dtype=torch.float64)
    xm, ym = xs.mean(), ys.mean()
    var = float(((xs - xm) ** 2).sum())
    slope = float(((xs - xm) * (ys - ym)).sum() / var) if var > 0 else 0.0
    icpt = float(ym - slope * xm)
    full_rows = [M + i for i in range(1, args.steps + 1)]
    t_budget = float(sum(us)) * 1e-3
    t_full = float(sum(icpt + slope * r for r in full_rows)) * 1e-3

    L, d = cfg.layers, cfg.q_heads * cfg.head_dim
    attn = lambda S: 4 * L * d * S                                           # Appendix A, per step
    mlp = 6 * d * d + d
    uses_mlp = preset.score_kind in ("predictor", "negated")
    flops_budget = sum(attn(r) for r in rows_at_step) + (mlp * args.steps if uses_mlp else 0)
    flops_full = sum(attn(r) for r in full_rows)
    pick = sorted(set(list(range(0, args.steps, max(1, args.steps // 24))) + [args.steps - 1]))
    res = {
        "preset": preset.name, "workload": cfg.name, "steps": args.steps, "B": B, "W_q": preset.n_pinned, "W_l": preset.window,
        "ratio": preset.ratio, "K_evicted_per_event": K, "events_measured": run.events, "events_closed_form": n_closed,
        "lengths_equal_closed_form": measured == closed,
        "sawtooth_step_measured_closed": [[i + 1, measured[i], closed[i]] for i in pick],
        "length_min_max_after_first_event": [min(measured[B - M - 1:]) if args.steps > B - M else None,
                                             max(measured[B - M - 1:]) if args.steps > B - M else None],
        "decode_us_per_step": {"mean": round(sum(us) / len(us), 2), "fit_us_per_row": round(slope, 5), "fit_intercept_us": round(icpt, 2)},
        "attention_time_ms": {"budget_measured": round(t_budget, 2), "full_kv_from_fit": round(t_full, 2),
                              "ratio": round(t_full / t_budget, 3) if t_budget > 0 else None},
        "flops_appendix_a": {"budget_attention_plus_predictor": flops_budget, "full_kv_attention": flops_full,
                             "ratio": round(flops_full / flops_budget, 3),
                             "eq9_net_saving_at_last_step": run.events * 4 * L * d * K - (mlp if uses_mlp else 0)},
        "data": "synthetic",
    }
    run.close()
    print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
