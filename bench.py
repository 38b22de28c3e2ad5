#!/usr/bin/env python
"""Benchmark of the decode hot path: fused decode attention + importance accumulation every
step, eviction + compaction every E steps, on a steady-state budget-limited KV cache.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2_llama8b] [--impl ours|reference]

A step is one decode step of the whole stack (all layers) for the whole batch; every
evict_interval-th step is followed by an eviction down to the budget.  Rank 0 prints one JSON
line.  With N > 1 (torchrun) every rank runs an independent replica of the workload: the path
has no exchange step, so there is no collective on the data path ("replicas only").
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402
from workloads import gen  # noqa: E402

METRIC = "decode tokens/s at budget B"
UNIT = "tokens/s"
BYTES_PER_SLOT = 520          # K row 256 + V row 256 + fp32 score read-modify-write 8 (bf16 d=128, fp32 d=64)
# DRAM bytes moved per algorithmic byte by the decode kernel, from the ncu capture summarised in
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum of one launch / its algorithmic bytes).
NCU_TRAFFIC_RATIO = 1.067


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.times, self.reasons, self.max_mhz = [], [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.times.append(time.perf_counter())
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def rank_seed(cfg, rank):
    """Seed of a rank's synthetic cache: every rank holds its own batch of the workload (independent
    sequences, sharded over the ranks with no exchange between them)."""
    return 1000 * int(cfg.name[1]) + rank


def max_over_ranks(x, world, device=None):
    """The slowest rank's time: what the whole job took (an all-reduce over the process group; the
    only collective of the benchmark, and none of the data path's)."""
    if world == 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(batch, steps, world, seconds):
    """Tokens per second of the whole job: every rank decodes `batch` sequences for `steps` steps."""
    return batch * steps * world / seconds


def workload_config(cfg, args, world):
    """The `config` object of the JSON line: a description of the workload that both arms print
    alike (nothing in it depends on which implementation ran)."""
    kv8 = args.kv_dtype == "fp8"
    elt = 1 if kv8 else (2 if cfg.dtype == "bf16" else 4)
    kv_bytes = cfg.layers * cfg.batch * cfg.kv_heads * cfg.capacity * 2 * cfg.head_dim * elt
    return {"workload": cfg.name, "layers": cfg.layers, "batch": cfg.batch, "q_heads": cfg.q_heads,
            "kv_heads": cfg.kv_heads, "head_dim": cfg.head_dim, "budget": cfg.budget, "window": cfg.window,
            "evict_interval": cfg.evict_interval, "prompt_pinned": cfg.prompt, "dist": cfg.dist,
            "score_source": args.score_source, "selection": args.selection,
            "kv_dtype": "e4m3 codes, scale 1/32" if kv8 else cfg.dtype,
            "kv_bytes": kv_bytes,
            "l2_policy": "inputs larger than L2 (K/V slabs %.0f MB vs 126 MB L2)" % (kv_bytes / 1e6),
            "replicas": world}


def setup_cache(cfg, seed, device, kv8=False, u=None):
    """A cache in steady state: every sequence holds `budget` rows (the prompt rows pinned).  u: the
    planted directions the decode queries will be aligned with (the fill's critical keys use them)."""
    import torch
    import paper_2601_18383_b200 as D
    cache = D.Cache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window,
                    cfg.evict_interval, dtype="bf16_kv8" if kv8 else cfg.dtype, seq_budgets=cfg.seq_budgets, device=device)
    if kv8:
        cache.set_kv_scale(1.0 / 32, 1.0 / 32)     # synthetic rows are O(1): well inside the format's range
    if cfg.seq_budgets:
        one = cfg.scaled(batch=1)
        for b in range(cfg.batch):
            k, v = gen.torch_keys_values(one, seed + b, cfg.seq_budgets[b], device, u=None if u is None else u[:, b:b + 1])
            cache.prefill_seq(b, k[:, 0], v[:, 0], n_pinned=cfg.prompt)
    else:
        k, v = gen.torch_keys_values(cfg, seed, cfg.budget, device, u=u)
        cache.prefill(k, v, n_pinned=cfg.prompt)
    del k, v
    torch.cuda.empty_cache()
    return cache


def slots_in_step(cfg, lens):
    return cfg.layers * cfg.kv_heads * sum(lens)


def run_ours(args, cfg, rank, world, device):
    import torch
    import torch.distributed as dist

    E = cfg.evict_interval
    ring_n = 64
    kv8 = args.kv_dtype == "fp8"
    if kv8 and (cfg.dtype != "bf16" or cfg.head_dim % 16):
        raise SystemExit("--kv-dtype fp8 needs a bf16 workload")
    seed = rank_seed(cfg, rank)
    # one set of planted directions for the steady-state fill and for the decode queries
    u = gen.torch_unit_dirs(cfg, seed, device) if cfg.dist == "planted" else None
    cache = setup_cache(cfg, seed, device, kv8, u=u)
    if args.evict_split:
        cache.set_evict_launch(args.evict_split)
    q_ring, k_ring, v_ring = gen.torch_step_ring(cfg, 77 + rank, ring_n, device, u=u)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=q_ring.dtype, device=device)
    stream = torch.cuda.current_stream(device)
    external = args.score_source == "external"
    bytes_per_slot = BYTES_PER_SLOT - 8 if external else BYTES_PER_SLOT   # no score read-modify-write
    if kv8:
        bytes_per_slot -= 2 * cfg.head_dim                                # K and V rows of head_dim bytes each
    if external:
        import paper_2601_18383_b200 as D
        cache.set_score_source(D.DYNTS_SCORE_EXTERNAL)
        g = torch.Generator(device=device).manual_seed(4242 + rank)
        s_ring = torch.randn((ring_n, cfg.batch), generator=g, device=device)   # stand-in for predictor outputs

    evict_call = cache.evict_global if args.selection == "global" else cache.evict
    peak, peak_kind = measured_peaks()
    elt = 1 if kv8 else (2 if cfg.dtype == "bf16" else 4)
    row_move_bytes = 2 * (2 * cfg.head_dim * elt + 8)      # K row + V row + pos + score, read and written

    def decode(j):
        cache.decode_attn(q_ring[j], k_ring[j], v_ring[j], out)
        if external:
            cache.append_scores(s_ring[j])

    state = {"since": 0, "i": 0, "evictions": 0}      # decode steps since the last eviction, kept across the phases below

    def step():
        decode(state["i"] % ring_n)
        state["i"] += 1
        state["since"] += 1
        if state["since"] == E:
            evict_call(0)
            state["since"] = 0
            state["evictions"] += 1

    def finish_cycle():
        while state["since"] != 0:
            step()

    def step_bytes():
        return bytes_per_slot * slots_in_step(cfg, [cache.len(bb) + 1 for bb in range(cfg.batch)])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    def event():
        return torch.cuda.Event(enable_timing=True)

    # warm-up: the requested steps rounded up to whole eviction cycles (at least one), so that scores and
    # selection are non-trivial and the timed region starts at the beginning of a cycle
    warm = max(args.warmup, 3)
    warm = (warm + E - 1) // E * E
    for _ in range(warm):
        step()
    barrier()
    cache.poll_error()

    # ---- timed region: exactly K steps, device-resident inputs --------------------------------
    K = args.steps
    sampler = ClockSampler(physical_gpu_index(torch.cuda.current_device()))
    sampler.start()
    launches0 = cache.launch_count()
    ev_before = state["evictions"]
    ev0, ev1 = event(), event()
    barrier()
    ev0.record(stream)
    for _ in range(K):
        step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    launches = cache.launch_count() - launches0
    evictions_in_region = state["evictions"] - ev_before
    cache.poll_error()
    ms = max_over_ranks(ms, world, device)
    value = job_throughput(cfg.batch, K, world, ms * 1e-3)

    # ---- per-kernel durations: whole eviction cycles, whatever K is -------------------------------
    # Every cycle is E back-to-back decode launches (one event pair around the run, so the average
    # launch duration includes the gaps between launches, as in the timed region) and the eviction
    # that follows (its own event pair).  At least 4 cycles, so at least 4 eviction events are timed.
    finish_cycle()
    n_cyc = max(4, min((K + E - 1) // E, 8))

    def timed_cycles(n):
        dec_runs, ev_events = [], []
        for _ in range(n):
            a, b, c = event(), event(), event()
            run_bytes = 0
            a.record(stream)
            for _j in range(E):
                run_bytes += step_bytes()
                decode(state["i"] % ring_n)
                state["i"] += 1
            b.record(stream)
            evict_call(0)
            c.record(stream)
            state["evictions"] += 1
            scanned, moved = cache.evict_stats()           # synchronises; outside the event pairs
            dec_runs.append((a, b, run_bytes))
            ev_events.append((b, c, 4 * scanned + row_move_bytes * moved, moved))
        torch.cuda.synchronize(device)
        cache.poll_error()
        return dec_runs, ev_events

    def evict_summary(ev_events):
        ev_ms = [a.elapsed_time(b) for a, b, _, _ in ev_events]
        ev_bytes = sum(x for _, _, x, _ in ev_events) / len(ev_events)
        ev_avg = sum(ev_ms) / len(ev_ms)
        ev_gbs = ev_bytes / (ev_avg * 1e-3) / 1e9 if ev_avg > 0 else 0.0
        return {"kernels": "evict (selection + in-place compaction, one launch)", "bound": "hbm", "achieved": round(ev_gbs, 1),
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": round(ev_gbs / peak, 4),
                "algorithmic_bytes_per_event": int(ev_bytes),
                "rows_moved_per_event": int(sum(m for _, _, _, m in ev_events) / len(ev_events)),
                "avg_event_us": round(1e3 * ev_avg, 2), "min_event_us": round(1e3 * min(ev_ms), 2),
                "evict_per_step_us": round(1e3 * ev_avg / E, 3), "events_timed": len(ev_ms),
                "decode_steps_before": state["i"]}, ev_avg, ev_bytes

    dec_runs, ev_events = timed_cycles(n_cyc)
    dec_launches = n_cyc * E
    dec_avg_ms = sum(a.elapsed_time(b) for a, b, _ in dec_runs) / dec_launches
    algo_bytes = sum(x for _, _, x in dec_runs) / dec_launches
    dec_gbs = algo_bytes / (dec_avg_ms * 1e-3) / 1e9
    roofline = {
        "kernel": "decode_attn (fused append + attention" + (" + append of the token's predictor score)" if external
                                                                 else " + importance accumulation)"),
        "bound": "hbm", "achieved": round(dec_gbs, 1), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
        "frac": round(dec_gbs / peak, 4),
        "traffic": None if (NCU_TRAFFIC_RATIO is None or external or kv8 or cfg.name != "c2_llama8b") else int(NCU_TRAFFIC_RATIO * algo_bytes),
        "algorithmic_bytes_per_launch": int(algo_bytes), "avg_launch_us": round(dec_avg_ms * 1e3, 2),
        "launches_timed": dec_launches,
    }
    evict, ev_avg, ev_bytes = evict_summary(ev_events)

    # ---- whole cycles without inner events: E decode steps + 1 eviction ----------------------------
    cyc = []
    for _ in range(n_cyc):
        a, c = event(), event()
        nbytes = 0
        a.record(stream)
        for _j in range(E):
            nbytes += step_bytes()
            decode(state["i"] % ring_n)
            state["i"] += 1
        evict_call(0)
        c.record(stream)
        state["evictions"] += 1
        cyc.append((a, c, nbytes))
    torch.cuda.synchronize(device)
    cyc_ms = sum(a.elapsed_time(c) for a, c, _ in cyc) / n_cyc
    cyc_bytes = sum(x for _, _, x in cyc) / n_cyc + ev_bytes
    cycle = {"decode_steps": E, "evictions": 1, "ms": round(cyc_ms, 4), "tokens_per_s": round(cfg.batch * E * world / (cyc_ms * 1e-3), 1),
             "algorithmic_bytes": int(cyc_bytes), "achieved": round(cyc_bytes / (cyc_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
             "frac": round(cyc_bytes / (cyc_ms * 1e-3) / 1e9 / peak, 4), "evict_share": round(ev_avg / cyc_ms, 4), "cycles_timed": n_cyc}

    # ---- sustained: whole cycles for at least args.sustain_seconds, clocks sampled throughout --------------
    sustained = evict_aged = None
    if args.sustain_seconds > 0:
        n_sus = max(2, int(args.sustain_seconds * 1e3 / cyc_ms) + 1)
        sus_sampler = ClockSampler(physical_gpu_index(torch.cuda.current_device()))
        marks = [event() for _ in range(n_sus + 1)]
        barrier()
        sus_sampler.start()
        t_start = time.perf_counter()
        marks[0].record(stream)
        for ci in range(n_sus):
            for _j in range(E):
                decode(state["i"] % ring_n)
                state["i"] += 1
            evict_call(0)
            state["evictions"] += 1
            marks[ci + 1].record(stream)
        barrier()
        sus_clk = sus_sampler.stop()
        ends = [marks[0].elapsed_time(m) for m in marks[1:]]            # ms since the start, on the device
        total_ms = ends[-1]
        total_ms = max_over_ranks(total_ms, world, device)
        # each cycle is attributed to the clock sample nearest to its middle, then binned by 50 MHz
        bins = {}
        if sus_sampler.samples:
            ts = np.asarray(sus_sampler.times) - t_start
            mhz = np.asarray(sus_sampler.samples, dtype=np.float64)
            prev = 0.0
            for e_ms in ends:
                mid = 0.5e-3 * (prev + e_ms)
                f = float(mhz[int(np.argmin(np.abs(ts - mid)))])
                key = int(round(f / 50.0) * 50)
                d = bins.setdefault(key, [0, 0.0])
                d[0] += 1
                d[1] += e_ms - prev
                prev = e_ms
        med = sus_clk["sm_mhz"]
        sustained = {"seconds": round(total_ms * 1e-3, 3), "cycles": n_sus, "steps": n_sus * E,
                     "tokens_per_s": round(cfg.batch * n_sus * E * world / (total_ms * 1e-3), 1),
                     "ms_per_step": round(total_ms / (n_sus * E), 5),
                     "clocks": sus_clk,
                     "step_us_x_sm_ghz": None if not med else round(total_ms * 1e3 / (n_sus * E) * med * 1e-3, 3),
                     "by_sm_mhz": [{"sm_mhz": k_, "cycles": v_[0], "tokens_per_s": round(cfg.batch * v_[0] * E * world / (v_[1] * 1e-3), 1)}
                                   for k_, v_ in sorted(bins.items())]}
        cache.poll_error()
        # the same eviction measurement on the aged cache: which rows an event evicts, and so how many
        # rows it moves, changes as the steady-state fill is replaced by decoded rows
        evict_aged = evict_summary(timed_cycles(4)[1])[0]

    # ---- end to end through the host-buffer entry point: whole cycles, evictions included ---------
    e2e = None
    if rank == 0 or world > 1:
        Ke = min(max(K, E), 4 * E)
        Ke = (Ke + E - 1) // E * E                     # whole cycles: every E-th step is followed by its eviction
        hq = [q_ring[j].cpu().pin_memory() for j in range(ring_n)]
        hk = [k_ring[j].cpu().pin_memory() for j in range(ring_n)]
        hv = [v_ring[j].cpu().pin_memory() for j in range(ring_n)]
        hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        for i in range(3):                             # warm-up of the entry point (staging set-up), then back to a cycle start
            cache.decode_attn_host(hq[i], hk[i], hv[i], hout)
        state["since"] = 3
        finish_cycle()
        barrier()
        t0 = time.perf_counter()
        e2e_evictions = 0
        for i in range(Ke):
            cache.decode_attn_host(hq[i % ring_n], hk[i % ring_n], hv[i % ring_n], hout)   # returns when `out` is on the host
            if (i + 1) % E == 0:
                evict_call(0)
                e2e_evictions += 1
        torch.cuda.synchronize(device)
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, world, device)
        e2e = {"value": round(job_throughput(cfg.batch, Ke, world, dt), 1), "unit": UNIT,
               "h2d_bytes_per_step": int(hq[0].numel() * hq[0].element_size() + 2 * hk[0].numel() * hk[0].element_size()),
               "d2h_bytes_per_step": int(hout.numel() * hout.element_size()), "steps": Ke, "evictions": e2e_evictions,
               "api": "dynts_decode_attn_host every step + dynts_evict every %d steps" % E}
        cache.poll_error()

    # ---- Importance Predictor head (Section 4.1): d -> 2d -> d/2 -> 1 at Llama-8B width -----------
    predictor = None
    if rank == 0 and world == 1 and not args.no_extras:
        predictor = time_predictor(cfg.batch, device, peak)

    # ---- prefill attention of the prompt (dense: tensor-bound) ------------------------------------
    prefill = None
    if rank == 0 and world == 1 and cfg.dtype == "bf16" and cfg.head_dim == 128 and not args.no_extras:
        prefill = time_prefill(cfg, device)
        prefill["long_prompt"] = {k: v for k, v in time_prefill(cfg, device, prompt=4096).items()
                                  if k in ("prompt_tokens", "layers_timed", "us_per_call", "flops", "achieved", "frac")}

    # ---- CPU baseline: the oracle, as it stands, on this machine's host cores (rank 0, N = 1) ------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not kv8:
        cpu = oracle_baseline(cfg, cache, q_ring, k_ring, v_ring, budget_s=args.cpu_seconds)

    config = workload_config(cfg, args, world)
    result = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
        "ms_per_step": round(ms / K, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": config,
        "run": {"warmup_steps_run": warm, "evictions_in_timed_region": evictions_in_region, "cache_bytes": cache.nbytes,
                "accumulate": "fp32 (softmax, output, scores)"},
        "hbm_gbs_decode": round(dec_gbs, 1), "roofline": roofline, "evict": evict, "evict_aged": evict_aged, "cycle": cycle, "sustained": sustained,
        "e2e": e2e, "predictor_mlp": predictor, "prefill_attn": prefill, "cpu_baseline": cpu, "clocks": clocks,
        "gpu_launches": int(launches),
    }
    cache.close()
    return result


def time_predictor(batch, device, peak, d=4096, iters=40):
    """Times dynts_predictor_mlp (three launches) on random bf16 weights; two weight sets alternate so
    that the 101 MB of weights are not served from L2."""
    import torch
    import paper_2601_18383_b200 as D
    g = torch.Generator(device=device).manual_seed(99)
    mk = lambda *shape: (torch.randn(shape, generator=g, device=device) / shape[-1] ** 0.5).to(torch.bfloat16)
    sets = [(mk(2 * d, d), mk(d // 2, 2 * d), mk(1, d // 2)) for _ in range(2)]
    h = torch.randn((batch, d), generator=g, device=device).to(torch.bfloat16)
    nbytes = D.dynts_predictor_mlp_scratch_bytes(d, batch)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=device)
    scores = torch.empty(batch, dtype=torch.float32, device=device)
    st = torch.cuda.current_stream(device)

    def run(i):
        W1, W2, W3 = sets[i % 2]
        D.dynts_predictor_mlp(h, W1, None, W2, None, W3, None, d, batch, 1, scratch, nbytes, scores, st.cuda_stream)

    for i in range(4):
        run(i)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(st)
    for i in range(iters):
        run(i)
    b.record(st)
    torch.cuda.synchronize(device)
    us = a.elapsed_time(b) * 1e3 / iters
    wbytes = 2 * (2 * d * d + d * d + d // 2)            # the bf16 weights, read once
    gbs = wbytes / (us * 1e-6) / 1e9
    return {"d": d, "batch": batch, "us_per_call": round(us, 2), "weight_bytes": wbytes, "bound": "hbm",
            "achieved": round(gbs, 1), "peak": peak, "unit": "GB/s", "frac": round(gbs / peak, 4)}


def time_prefill(cfg, device, iters=10, prompt=None):
    """Times the prompt attention (dynts_prompt_attn: Eq. 4-5 over the workload's prompt, all heads of
    up to 8 layers; the fill of the slabs is not part of it); flops = 4 d per (query, key) pair of the
    causal triangle; peak = the measured dense bf16 GEMM rate.  With `prompt`, the same heads on a
    prompt of that length, the batch shrunk to keep the token count (the long-prompt regime, where the
    per-tile rate shows rather than the fill and drain of the short items)."""
    import torch
    import paper_2601_18383_b200 as D
    sub = cfg.scaled(layers=min(cfg.layers, 8), seq_budgets=None, budget=max(cfg.budget, cfg.prompt))
    if prompt is not None:
        batch = max(1, min(cfg.batch, cfg.batch * cfg.prompt // prompt))
        sub = sub.scaled(prompt=prompt, batch=batch, budget=max(cfg.budget, prompt))
    T = sub.prompt
    cache = D.Cache(sub.layers, sub.batch, sub.q_heads, sub.kv_heads, sub.head_dim, sub.budget, sub.window, sub.evict_interval,
                    dtype="bf16", device=device)
    g = torch.Generator(device=device).manual_seed(7)
    q = torch.randn((sub.layers, sub.batch, sub.q_heads, T, 128), generator=g, device=device).to(torch.bfloat16)
    k, v = gen.torch_keys_values(sub, 9, T, device)
    out = torch.empty_like(q)
    st = torch.cuda.current_stream(device)
    for _ in range(3):
        cache.prompt_attn(q, k, v, out)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(st)
    for _ in range(iters):
        cache.prompt_attn(q, k, v, out)
    b.record(st)
    torch.cuda.synchronize(device)
    cache.poll_error()
    us = a.elapsed_time(b) * 1e3 / iters
    cache.close()
    flops = 4 * 128 * (T * (T + 1) // 2) * sub.layers * sub.batch * sub.q_heads
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak_tf, kind = float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        peak_tf, kind = 1590.0, "fallback"
    tf = flops / (us * 1e-6) / 1e12
    return {"kernel": "prefill_attn (tcgen05.mma, accumulators in tensor memory, TMA operands)", "prompt_tokens": T,
            "layers_timed": sub.layers, "us_per_call": round(us, 1), "flops": flops, "bound": "tensor",
            "achieved": round(tf, 1), "peak": peak_tf, "peak_kind": kind, "unit": "TFLOP/s", "frac": round(tf / peak_tf, 4)}


def oracle_baseline(cfg, cache, q_ring, k_ring, v_ring, budget_s=20.0, slabs=None):
    """Times oracle decode steps (and one eviction) on a bounded sample of the same workload: the
    state of a subset of layers is exported from the device cache; throughput is scaled by the
    fraction of slabs processed."""
    import torch
    from oracle import dynts_oracle as O
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    # sample: layer 0 of every sequence and KV head (exported from the device cache)
    total_slabs = cfg.layers * cfg.batch * cfg.kv_heads
    nl = 1
    orc = O.OracleCache(nl, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.window, cache.capacity)
    for b in range(cfg.batch):
        for h in range(cfg.kv_heads):
            K, V, pos, score = cache.export_slab(0, b, h)
            s = orc.slab(0, b, h)
            n = K.shape[0]
            if n >= cache.capacity:
                n = cache.capacity - 1
            s.K[:n], s.V[:n] = K[:n].double().numpy(), V[:n].double().numpy()
            s.pos[:n], s.score[:n], s.n = pos[:n].numpy(), score[:n].double().numpy(), n
        orc.n_pinned[b] = cfg.prompt
    q = q_ring[:, :nl].double().cpu().numpy()
    k = k_ring[:, :nl].double().cpu().numpy()
    v = v_ring[:, :nl].double().cpu().numpy()
    t0 = time.perf_counter()
    steps = 0
    while time.perf_counter() - t0 < budget_s and steps < 65536:
        if any(orc.slab(0, b, 0).n + 1 > cache.capacity for b in range(cfg.batch)):
            O.evict(orc, list(cfg.seq_budgets) if cfg.seq_budgets else cfg.budget)
        j = steps % q.shape[0]
        O.decode_step(orc, q[j], k[j], v[j])
        steps += 1
    dt = time.perf_counter() - t0
    frac = (nl * cfg.batch * cfg.kv_heads) / total_slabs
    value = cfg.batch * steps / dt * frac
    return {"value": round(value, 3), "unit": UNIT, "cores": int(threads), "kind": "oracle",
            "sample": f"{steps} decode steps (+ evictions as they fall due) over layer 0 of {cfg.layers} "
                      f"({nl * cfg.batch * cfg.kv_heads} of {total_slabs} slabs) in {dt:.1f} s; scaled by the slab fraction"}


def run_reference(args, cfg, rank, world):
    """The reference arm is the float64 oracle on the host cores (rank 0 only)."""
    if rank != 0:
        return None
    from oracle import dynts_oracle as O
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    total_slabs = cfg.layers * cfg.batch * cfg.kv_heads
    # calibrate one slab-step, then size the per-step sample so the whole run stays within ~2 min
    one = cfg.scaled(layers=1, batch=1, kv_heads=1, q_heads=cfg.group, seq_budgets=None)
    pk, pv = W.prompt_kv(one, 5, n_tokens=cfg.budget)
    orc = O.OracleCache(1, 1, cfg.group, 1, cfg.head_dim, cfg.window, cfg.capacity)
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64), n_pinned=cfg.prompt)
    st = W.DecodeStream(one, 5)
    t0 = time.perf_counter()
    for s in range(1, 4):
        q, k, v = st.step(s)
        O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
    per_slab = (time.perf_counter() - t0) / 3
    steps_total = args.steps + args.warmup
    n_slabs = int(max(1, min(total_slabs, 100.0 / max(per_slab * steps_total, 1e-9))))
    heads = min(cfg.kv_heads, n_slabs)
    seqs = max(1, min(cfg.batch, n_slabs // heads))
    layers = max(1, min(cfg.layers, n_slabs // (heads * seqs)))
    sub = cfg.scaled(layers=layers, batch=seqs, kv_heads=heads, q_heads=heads * cfg.group,
                     seq_budgets=cfg.seq_budgets[:seqs] if cfg.seq_budgets else None)
    used = layers * seqs * heads
    pk, pv = W.prompt_kv(sub, 6, n_tokens=min(sub.seq_budgets) if sub.seq_budgets else sub.budget)
    orc = O.OracleCache(layers, seqs, sub.q_heads, heads, cfg.head_dim, cfg.window, cfg.capacity)
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64), n_pinned=cfg.prompt)
    st = W.DecodeStream(sub, 6)
    ring = [tuple(x.astype(np.float64) for x in st.step(s)) for s in range(1, 9)]
    tgt = list(sub.seq_budgets) if sub.seq_budgets else sub.budget

    def step(i):
        O.decode_step(orc, *ring[i % len(ring)])
        if (i + 1) % cfg.evict_interval == 0:
            O.evict(orc, tgt)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    value = cfg.batch * args.steps / dt * (used / total_slabs)
    sample = (f"each step = one oracle decode step (eviction every {cfg.evict_interval}) over {used} of {total_slabs} "
              f"slabs ({layers} layers x {seqs} sequences x {heads} KV heads); throughput scaled by that fraction")
    return {
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3 * (total_slabs / used), 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args, world),
        "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": int(threads), "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8192)
    ap.add_argument("--warmup", type=int, default=128)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_llama8b", choices=sorted(W.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--sustain-seconds", type=float, default=2.0,
                    help="length of the sustained region that follows the K timed steps (0: skip it)")
    ap.add_argument("--no-extras", action="store_true", help="skip the predictor-head and prefill-attention timings")
    ap.add_argument("--extras-only", action="store_true",
                    help="time only the predictor head and the prefill attention of the workload (a short run, e.g. to profile them)")
    ap.add_argument("--score-source", default="attention", choices=["attention", "external"],
                    help="attention: Eq. 6 mass accumulated online (default); external: one predictor score per token (Eq. 7)")
    ap.add_argument("--selection", default="slab", choices=["slab", "global"],
                    help="slab: every (layer, KV head) selects on its own scores; global: one selection per sequence")
    ap.add_argument("--kv-dtype", default="bf16", choices=["bf16", "fp8"],
                    help="fp8: the slabs hold E4M3 codes (q, k, v, out stay bf16); bf16 workloads only")
    ap.add_argument("--evict-split", type=int, default=0, help="CTAs per slab of the eviction kernel (0: automatic; tuning)")
    ap.add_argument("--cluster", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0)
    args = ap.parse_args()
    cfg = W.get_config(args.workload)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        res = run_reference(args, cfg, rank, world)
        if res is not None:
            print(json.dumps(res), flush=True)
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    if args.cluster or args.variant:
        import paper_2601_18383_b200 as D
        _orig = D.Cache.__init__

        def _init(self, *a, **kw):
            _orig(self, *a, **kw)
            self.set_launch(args.cluster, args.variant)
        D.Cache.__init__ = _init
    if args.extras_only:
        peak, _ = measured_peaks()
        res = {"config": workload_config(cfg, args, world), "predictor_mlp": time_predictor(cfg.batch, device, peak),
               "prefill_attn": time_prefill(cfg, device) if cfg.dtype == "bf16" and cfg.head_dim == 128 else None}
        if res["prefill_attn"]:
            res["prefill_attn"]["long_prompt"] = time_prefill(cfg, device, prompt=4096)
    else:
        res = run_ours(args, cfg, rank, world, device)
    if rank == 0:
        print(json.dumps(res), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
