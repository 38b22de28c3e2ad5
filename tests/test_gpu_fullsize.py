"""Full-size checks in the launch configuration the benchmark times (automatic cluster size and
kernel variant): steady-state caches of the stated shapes are filled on the device from a seeded
generator; sampled slabs are exported and the oracle recomputes them one by one."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads import gen
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _steady_state(cfg, seed, rows):
    gpu = H.make_gpu(cfg)
    k, v = gen.torch_keys_values(cfg, seed, rows, "cuda:0")
    gpu.prefill(k, v, n_pinned=cfg.prompt)
    del k, v
    return gpu


def _check_sampled(gpu, cfg, seed, slabs, steps=3):
    ring = gen.torch_step_ring(cfg, seed, steps, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=H.tdtype(cfg), device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    worst = dict(out=0.0, delta=0.0)
    for s in range(steps):
        orc = H.oracle_from_gpu(gpu, cfg, slabs=slabs)
        q, k, v = ring[0][s], ring[1][s], ring[2][s]
        gpu.decode_attn(q, k, v, out, delta)
        gpu.synchronize()
        gpu.poll_error()
        qh, kh, vh = q.double().cpu().numpy(), k.double().cpu().numpy(), v.double().cpu().numpy()
        og, dh = out.float().cpu().numpy(), delta.cpu().numpy()
        G = cfg.group
        for (l, b, h) in slabs:
            sl = orc.slab(l, b, h)
            sl.K[sl.n], sl.V[sl.n] = kh[l, b, h], vh[l, b, h]
            n = sl.n + 1
            alpha = O.attention_weights(qh[l, b, h * G:(h + 1) * G], sl.K[:n])
            o_ref = O.attention_output(alpha, sl.V[:n])
            worst["out"] = max(worst["out"], H.rel_err_vectors(og[l, b, h * G:(h + 1) * G], o_ref))
            worst["delta"] = max(worst["delta"], float(np.abs(dh[l, b, h, :n] - alpha.sum(axis=0)).max()))
    return worst


def _sample_slabs(cfg, k, seed):
    r = np.random.default_rng(seed)
    all_ = [(l, b, h) for l in range(cfg.layers) for b in range(cfg.batch) for h in range(cfg.kv_heads)]
    idx = r.choice(len(all_), size=min(k, len(all_)), replace=False)
    return [all_[i] for i in idx] + [all_[0], all_[-1]]


def test_config2_full_size():
    cfg = W.get_config("c2_llama8b")
    gpu = _steady_state(cfg, 2100, cfg.budget + 5)
    slabs = _sample_slabs(cfg, 10, 1)
    worst = _check_sampled(gpu, cfg, 2100, slabs, steps=cfg.evict_interval - 5 - 2)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    # run up to the eviction point with the accumulated (non-trivial) scores, then evict
    ring = gen.torch_step_ring(cfg, 2101, 2, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    for s in range(2):
        gpu.decode_attn(ring[0][s], ring[1][s], ring[2][s], out)
    assert gpu.len(0) == cfg.capacity
    H.check_evict_bit_exact(gpu, cfg, 0, slabs=slabs)
    assert gpu.len(0) == cfg.budget
    worst = _check_sampled(gpu, cfg, 2102, slabs, steps=2)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    gpu.close()


def test_config3_full_size():
    cfg = W.get_config("c3_qwen7b")
    gpu = _steady_state(cfg, 3100, cfg.capacity - 3)
    slabs = _sample_slabs(cfg, 8, 2)
    worst = _check_sampled(gpu, cfg, 3100, slabs, steps=3)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    assert gpu.len(0) == cfg.capacity
    H.check_evict_bit_exact(gpu, cfg, 0, slabs=slabs)
    assert gpu.len(15) == cfg.budget
    gpu.close()
    torch.cuda.empty_cache()


def test_config4_full_size_ragged():
    cfg = W.get_config("c4_ragged")
    gpu = H.make_gpu(cfg)
    one = cfg.scaled(batch=1)
    r = np.random.default_rng(4100)
    rows = []
    for b in range(cfg.batch):
        n = int(cfg.seq_budgets[b] + r.integers(1, cfg.evict_interval - 2))
        k, v = gen.torch_keys_values(one, 4100 + b, n, "cuda:0")
        gpu.prefill_seq(b, k[:, 0], v[:, 0], n_pinned=cfg.prompt)
        rows.append(n)
    assert [gpu.len(b) for b in range(cfg.batch)] == rows
    slabs = _sample_slabs(cfg, 10, 3)
    worst = _check_sampled(gpu, cfg, 4100, slabs, steps=2)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    H.check_evict_bit_exact(gpu, cfg, 0, slabs=slabs)
    assert [gpu.len(b) for b in range(cfg.batch)] == list(cfg.seq_budgets)
    gpu.close()
    torch.cuda.empty_cache()


def test_config5_attention_shapes_layer_by_layer():
    """The attention part of the full-model configuration (32 layers, 32/8 heads, batch 8, budget
    3072), driven the way a model drives it: one call per layer.  Window 128 and interval 64 are
    the reading taken here (the configuration names neither)."""
    cfg = W.get_config("c2_llama8b").scaled(name="c5_attn", batch=8, budget=3072, window=128, evict_interval=64,
                                             prompt=256, density=0.03)
    gpu = _steady_state(cfg, 5100, cfg.capacity - 2)
    slabs = _sample_slabs(cfg, 10, 5)
    ring = gen.torch_step_ring(cfg, 5100, 2, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    G = cfg.group
    for s in range(2):
        orc = H.oracle_from_gpu(gpu, cfg, slabs=slabs)
        q, k, v = ring[0][s], ring[1][s], ring[2][s]
        for l in range(cfg.layers):
            gpu.decode_attn_layer(l, q[l], k[l], v[l], out[l], delta)
        gpu.synchronize()
        gpu.poll_error()
        qh, kh, vh = q.double().cpu().numpy(), k.double().cpu().numpy(), v.double().cpu().numpy()
        og, dh = out.float().cpu().numpy(), delta.cpu().numpy()
        for (l, b, h) in slabs:
            sl = orc.slab(l, b, h)
            sl.K[sl.n], sl.V[sl.n] = kh[l, b, h], vh[l, b, h]
            n = sl.n + 1
            alpha = O.attention_weights(qh[l, b, h * G:(h + 1) * G], sl.K[:n])
            o_ref = O.attention_output(alpha, sl.V[:n])
            assert H.rel_err_vectors(og[l, b, h * G:(h + 1) * G], o_ref) <= H.TOL_OUT["bf16"]
            assert float(np.abs(dh[l, b, h, :n] - alpha.sum(axis=0)).max()) <= H.TOL_DELTA
    assert gpu.len(0) == cfg.capacity
    H.check_evict_bit_exact(gpu, cfg, 0, slabs=slabs)
    assert gpu.len(7) == cfg.budget
    gpu.close()
    torch.cuda.empty_cache()


def test_full_kv_length_slabs_and_two_kernel_eviction():
    """The longest slabs the configurations name (full KV of the 16384-token decode: 16640 rows):
    the streaming kernel spreads every slab over many CTAs, and the eviction takes the two-kernel
    path (gather list in global memory) because such a slab does not fit the fused kernel."""
    cfg = W.get_config("c2_llama8b").scaled(name="full_kv", layers=2, batch=2, budget=16640, window=128, evict_interval=64,
                                             prompt=256, density=0.01)
    gpu = _steady_state(cfg, 6100, 16640 - 2)
    slabs = [(0, 0, 0), (1, 1, 7), (0, 1, 3)]
    worst = _check_sampled(gpu, cfg, 6100, slabs, steps=2)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    assert gpu.len(0) == 16640
    H.check_evict_bit_exact(gpu, cfg, 12000, slabs=slabs)
    assert gpu.len(1) == 12000
    worst = _check_sampled(gpu, cfg, 6101, slabs, steps=1)
    assert worst["out"] <= H.TOL_OUT["bf16"] and worst["delta"] <= H.TOL_DELTA, worst
    gpu.close()
    torch.cuda.empty_cache()


def test_an_eviction_cycle_replays_as_a_cuda_graph():
    """E decode steps and the eviction that follows return the cache to the same lengths, so the
    cycle can be captured once and replayed; the replayed state must equal the eagerly run one."""
    cfg = W.get_config("c2_llama8b").scaled(layers=4, batch=2, prompt=64, budget=512, window=32, evict_interval=16)
    E = cfg.evict_interval
    caches = []
    for _ in range(2):
        g = H.make_gpu(cfg)
        k, v = gen.torch_keys_values(cfg, 7100, cfg.budget, "cuda:0")
        g.prefill(k, v, n_pinned=cfg.prompt)
        caches.append(g)
    a, b = caches
    q, kk, vv = gen.torch_step_ring(cfg, 7100, E, "cuda:0")
    oa = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    ob = torch.empty_like(oa)

    def cycle(c, o):
        for s in range(E):
            c.decode_attn(q[s], kk[s], vv[s], o)
        c.evict(0)

    cycle(a, oa)
    cycle(b, ob)                      # warm-up outside the capture (first-call set-up)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        b.set_stream(side)
        with torch.cuda.graph(graph, stream=side):
            cycle(b, ob)
    b.set_stream(torch.cuda.current_stream())
    torch.cuda.synchronize()
    # the capture ran nothing: b is one cycle behind a; replay twice, run a twice more eagerly
    cycle(a, oa)
    cycle(a, oa)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    a.poll_error(); b.poll_error()
    assert a.len(0) == b.len(0) == cfg.budget
    assert torch.equal(oa.view(torch.int16), ob.view(torch.int16))
    for l, bb, h in [(0, 0, 0), (3, 1, 7), (2, 0, 5)]:
        Ka, Va, pa, sa = a.export_slab(l, bb, h)
        Kb, Vb, pb, sb = b.export_slab(l, bb, h)
        assert torch.equal(pa, pb) and torch.equal(H.bits(sa), H.bits(sb)) and torch.equal(H.bits(Ka), H.bits(Kb))
    a.close(); b.close()


def test_two_caches_on_two_streams_do_not_interfere():
    """Two caches of different shapes driven alternately on their own streams (their kernels may
    overlap on the GPU) give bit-identical results to the same caches driven one after the other."""
    cfgs = [W.get_config("c2_llama8b").scaled(layers=6, batch=3, prompt=64, budget=448, window=32, evict_interval=16),
            W.get_config("c3_qwen7b").scaled(layers=4, batch=2, kv_heads=2, q_heads=14, prompt=48, budget=320, window=16,
                                            evict_interval=16)]
    results = []
    for mode in ("interleaved", "sequential"):
        caches, rings, outs, streams = [], [], [], []
        for i, cfg in enumerate(cfgs):
            g = H.make_gpu(cfg)
            k, v = gen.torch_keys_values(cfg, 8100 + i, cfg.budget, "cuda:0")
            g.prefill(k, v, n_pinned=cfg.prompt)
            caches.append(g)
            rings.append(gen.torch_step_ring(cfg, 8100 + i, 16, "cuda:0"))
            outs.append(torch.zeros((cfg.layers, cfg.batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0"))
            streams.append(torch.cuda.Stream())
        torch.cuda.synchronize()
        if mode == "interleaved":
            for i, g in enumerate(caches):
                g.set_stream(streams[i])
        order = [(s, i) for s in range(48) for i in range(2)] if mode == "interleaved" else \
                [(s, i) for i in range(2) for s in range(48)]
        for s, i in order:
            q, kk, vv = rings[i]
            caches[i].decode_attn(q[s % 16], kk[s % 16], vv[s % 16], outs[i])
            if (s + 1) % 16 == 0:
                caches[i].evict(0)
        torch.cuda.synchronize()
        snap = []
        for i, g in enumerate(caches):
            g.poll_error()
            cfg = cfgs[i]
            K, V, pos, score = g.export_slab(cfg.layers - 1, cfg.batch - 1, cfg.kv_heads - 1)
            snap.append((outs[i].clone(), K, pos, score))
            g.close()
        results.append(snap)
    for a, b in zip(*results):
        assert torch.equal(a[0].view(torch.int16), b[0].view(torch.int16))
        assert torch.equal(H.bits(a[1]), H.bits(b[1])) and torch.equal(a[2], b[2]) and torch.equal(H.bits(a[3]), H.bits(b[3]))


def test_config2_scores_when_the_last_pass_moves_into_the_next_launch():
    """Decode steps that do not ask for the step's mass, on equally long slabs that fill the grid:
    the launch then leaves the score pass of every CTA's last slab to the next launch.  The scores
    read back (which applies what is still recorded) must equal the oracle's after every read, in
    the middle of the run, after the run and across an eviction."""
    cfg = W.get_config("c2_llama8b")
    gpu = _steady_state(cfg, 2300, cfg.budget + 3)
    slabs = _sample_slabs(cfg, 6, 3)
    orc = H.oracle_from_gpu(gpu, cfg, slabs=slabs)
    steps = 24
    ring = gen.torch_step_ring(cfg, 2300, steps, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    G = cfg.group
    launches0 = gpu.launch_count()
    for s in range(steps):
        q, k, v = ring[0][s], ring[1][s], ring[2][s]
        gpu.decode_attn(q, k, v, out)
        qh, kh, vh = q.double().cpu().numpy(), k.double().cpu().numpy(), v.double().cpu().numpy()
        for (l, b, h) in slabs:
            sl = orc.slab(l, b, h)
            sl.K[sl.n], sl.V[sl.n], sl.score[sl.n] = kh[l, b, h], vh[l, b, h], 0.0
            sl.n += 1
            alpha = O.attention_weights(qh[l, b, h * G:(h + 1) * G], sl.K[:sl.n])
            sl.score[:sl.n] += alpha.sum(axis=0)
            if s in (6, steps - 1):
                o_ref = O.attention_output(alpha, sl.V[:sl.n])
                assert H.rel_err_vectors(out.float().cpu().numpy()[l, b, h * G:(h + 1) * G], o_ref) <= H.TOL_OUT["bf16"]
        if s in (6, steps - 1):
            sc = gpu.scores_tensor().cpu().numpy()
            for (l, b, h) in slabs:
                sl = orc.slab(l, b, h)
                fin = np.isfinite(sl.score[:sl.n])
                assert np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max() <= H.TOL_DELTA, (s, l, b, h)
    # one launch per step plus the two that applied the recorded passes when the scores were read
    assert gpu.launch_count() - launches0 == steps + 2
    gpu.poll_error()
    while gpu.len(0) < cfg.capacity:
        gpu.decode_attn(ring[0][0], ring[1][0], ring[2][0], out)
    H.check_evict_bit_exact(gpu, cfg, 0, slabs=slabs)
    assert gpu.len(0) == cfg.budget
    gpu.close()


@pytest.mark.parametrize("every", [2, 3])
def test_recorded_pass_on_short_slabs(every):
    """The same hand-over on slabs so short that a CTA finishes its slab before its scorer warp has
    applied the record of the previous launch: the new record must not be lost."""
    cfg = W.get_config("c2_llama8b").scaled(budget=256, window=16, evict_interval=64, prompt=32)
    gpu = _steady_state(cfg, 2400, cfg.budget + 3)
    slabs = [(0, 0, 0), (5, 0, 3), (31, 0, 7)]
    orc = H.oracle_from_gpu(gpu, cfg, slabs=slabs)
    ring = gen.torch_step_ring(cfg, 2400, 12, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    G = cfg.group
    for s in range(12):
        q, k, v = ring[0][s], ring[1][s], ring[2][s]
        gpu.decode_attn(q, k, v, out)
        qh, kh, vh = q.double().cpu().numpy(), k.double().cpu().numpy(), v.double().cpu().numpy()
        for (l, b, h) in slabs:
            sl = orc.slab(l, b, h)
            sl.K[sl.n], sl.V[sl.n], sl.score[sl.n] = kh[l, b, h], vh[l, b, h], 0.0
            sl.n += 1
            sl.score[:sl.n] += O.attention_weights(qh[l, b, h * G:(h + 1) * G], sl.K[:sl.n]).sum(axis=0)
        if (s + 1) % every == 0:
            sc = gpu.scores_tensor().cpu().numpy()
            for (l, b, h) in slabs:
                sl = orc.slab(l, b, h)
                fin = np.isfinite(sl.score[:sl.n])
                assert np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max() <= H.TOL_DELTA, (s, l, b, h)
    gpu.poll_error()
    gpu.close()


@pytest.mark.parametrize("kv8", [False, True])
def test_eviction_right_after_recorded_passes_equals_the_eager_path(kv8):
    """Two caches on the same inputs: one is asked for every step's mass (so every score pass runs
    inside its launch), the other is not (whole-slab pieces: the last pass of every CTA is recorded
    and, at the eviction, applied by the eviction kernel itself).  After the eviction both must hold
    the same bits: scores, positions, K, V."""
    import paper_2601_18383_b200 as D
    cfg = W.get_config("c2_llama8b").scaled(budget=256, window=16, evict_interval=32, prompt=32)
    caches = []
    for _ in range(2):
        g = D.Cache(cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, cfg.budget, cfg.window, cfg.evict_interval,
                    dtype="bf16_kv8" if kv8 else "bf16")
        if kv8:
            g.set_kv_scale(0.03125, 0.0625)
        k, v = gen.torch_keys_values(cfg, 2600, cfg.budget, "cuda:0")
        g.prefill(k, v, n_pinned=cfg.prompt)
        caches.append(g)
    eager, lazy = caches
    ring = gen.torch_step_ring(cfg, 2600, cfg.evict_interval, "cuda:0")
    oe = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    ol = torch.empty_like(oe)
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, eager.capacity), dtype=torch.float32, device="cuda:0")
    for cycle in range(2):
        for s in range(cfg.evict_interval):
            eager.decode_attn(ring[0][s], ring[1][s], ring[2][s], oe, delta)
            lazy.decode_attn(ring[0][s], ring[1][s], ring[2][s], ol)
        n0 = lazy.launch_count()
        eager.evict(0)
        lazy.evict(0)
        assert lazy.launch_count() - n0 == 1            # no separate launch for the recorded passes
        assert torch.equal(oe.view(torch.int16), ol.view(torch.int16))
        for sl in [(0, 0, 0), (7, 0, 3), (31, 0, 7), (16, 0, 5)]:
            Ke, Ve, pe, se = eager.export_slab(*sl)
            Kl, Vl, pl, sl_ = lazy.export_slab(*sl)
            assert torch.equal(pe, pl) and torch.equal(H.bits(se), H.bits(sl_)), (cycle, sl)
            assert torch.equal(H.bits(Ke), H.bits(Kl)) and torch.equal(H.bits(Ve), H.bits(Vl))
    eager.poll_error(); lazy.poll_error()
    eager.close(); lazy.close()


def _fill(cfg, gpu, seed):
    """Steady-state rows for every sequence: capacity - 3 rows (equal budgets) or, for a ragged
    batch, each sequence's budget plus a seeded number of rows below the eviction interval."""
    if cfg.seq_budgets:
        one = cfg.scaled(batch=1)
        r = np.random.default_rng(seed)
        for b in range(cfg.batch):
            n = int(cfg.seq_budgets[b] + r.integers(1, cfg.evict_interval - 3))
            k, v = gen.torch_keys_values(one, seed + b, n, "cuda:0")
            gpu.prefill_seq(b, k[:, 0], v[:, 0], n_pinned=cfg.prompt)
    else:
        k, v = gen.torch_keys_values(cfg, seed, cfg.capacity - 3, "cuda:0")
        gpu.prefill(k, v, n_pinned=cfg.prompt)


@pytest.mark.parametrize("name", ["c3_qwen7b", "c4_ragged"])
def test_the_benchmarks_exact_call_at_full_size(name):
    """decode_attn(..., scores = NULL) followed by evict, as bench.py issues them (config 3: whole-slab
    pieces of 7 slabs per CTA whose last score pass is recorded and applied by the next launch or by
    the eviction kernel; config 4: stream-K pieces over a ragged batch).  Sampled slabs against the
    oracle: outputs every step, accumulated scores in the middle of the run (Eq. 6).  The eviction
    is checked through a second cache on the same inputs that is asked for every step's mass, so
    that all its score passes run inside their launches: its eviction must equal the oracle's
    selection from its own float32 scores bit for bit (Section 4.2), and the first cache, evicted
    without any read in between, must hold the same bits."""
    cfg = W.get_config(name)
    lazy, eager = H.make_gpu(cfg), H.make_gpu(cfg)
    _fill(cfg, lazy, 8100)
    _fill(cfg, eager, 8100)
    slabs = _sample_slabs(cfg, 8, 11)
    orc = H.oracle_from_gpu(lazy, cfg, slabs=slabs)
    steps = 3
    ring = gen.torch_step_ring(cfg, 8100, steps, "cuda:0")
    ol = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    oe = torch.empty_like(ol)
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, eager.capacity), dtype=torch.float32, device="cuda:0")
    G = cfg.group
    for s in range(steps):
        q, k, v = ring[0][s], ring[1][s], ring[2][s]
        lazy.decode_attn(q, k, v, ol)                       # the benchmark's call
        eager.decode_attn(q, k, v, oe, delta)
        assert torch.equal(ol.view(torch.int16), oe.view(torch.int16))
        qh, kh, vh = q.double().cpu().numpy(), k.double().cpu().numpy(), v.double().cpu().numpy()
        og = ol.float().cpu().numpy()
        for (l, b, h) in slabs:
            sl = orc.slab(l, b, h)
            sl.K[sl.n], sl.V[sl.n], sl.score[sl.n] = kh[l, b, h], vh[l, b, h], 0.0
            sl.n += 1
            alpha = O.attention_weights(qh[l, b, h * G:(h + 1) * G], sl.K[:sl.n])
            sl.score[:sl.n] += alpha.sum(axis=0)
            o_ref = O.attention_output(alpha, sl.V[:sl.n])
            assert H.rel_err_vectors(og[l, b, h * G:(h + 1) * G], o_ref) <= H.TOL_OUT["bf16"], (s, l, b, h)
        if s == steps - 2:                                  # a read in the middle applies what is recorded
            sc = lazy.scores_tensor().cpu().numpy()
            for (l, b, h) in slabs:
                sl = orc.slab(l, b, h)
                fin = np.isfinite(sl.score[:sl.n])
                assert np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max() <= H.TOL_DELTA, (s, l, b, h)
            del sc
    lazy.poll_error()
    n0 = lazy.launch_count()
    lazy.evict(0)                                           # straight after the last decode launch
    assert lazy.launch_count() - n0 == 1
    lazy.synchronize()
    lazy.poll_error()
    # the eager cache: scores against the oracle, then its eviction against the oracle's selection
    sc = eager.scores_tensor().cpu().numpy()
    for (l, b, h) in slabs:
        sl = orc.slab(l, b, h)
        fin = np.isfinite(sl.score[:sl.n])
        assert np.abs(sc[l, b, h, :sl.n][fin] - sl.score[:sl.n][fin]).max() <= H.TOL_DELTA, (l, b, h)
    del sc
    H.check_evict_bit_exact(eager, cfg, 0, slabs=slabs)
    targets = list(cfg.seq_budgets) if cfg.seq_budgets else [cfg.budget] * cfg.batch
    assert [lazy.len(b) for b in range(cfg.batch)] == targets == [eager.len(b) for b in range(cfg.batch)]
    for sl in slabs:
        Ke, Ve, pe, se = eager.export_slab(*sl)
        Kl, Vl, pl, s_l = lazy.export_slab(*sl)
        assert torch.equal(pe, pl) and torch.equal(H.bits(se), H.bits(s_l)), sl
        assert torch.equal(H.bits(Ke), H.bits(Kl)) and torch.equal(H.bits(Ve), H.bits(Vl)), sl
    lazy.close()
    eager.close()
    torch.cuda.empty_cache()


def test_sequence_wide_selection_on_full_kv_length_slabs():
    """dynts_evict_global on slabs too long for the fused kernel (16640 rows): the two-kernel path
    ranks every slab by the keys shared across the sequence (Appendix B.1)."""
    cfg = W.get_config("c2_llama8b").scaled(name="full_kv_global", layers=2, batch=1, kv_heads=2, q_heads=8, budget=16640,
                                             window=128, evict_interval=64, prompt=256, density=0.01)
    gpu = _steady_state(cfg, 6200, 16640 - 2)
    ring = gen.torch_step_ring(cfg, 6200, 2, "cuda:0")
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    for s in range(2):
        gpu.decode_attn(ring[0][s], ring[1][s], ring[2][s], out)
    n = gpu.len(0)
    assert n == 16640
    keys_t = torch.zeros((cfg.batch, gpu.capacity), dtype=torch.float32, device="cuda:0")
    gpu.aggregate_scores(keys_t)
    keys = keys_t.cpu().numpy()
    sc = gpu.scores_tensor().cpu().numpy()
    exact = sc[:, 0, :, :n].astype(np.float64).sum(axis=(0, 1))
    fin = np.isfinite(exact)
    assert np.abs(keys[0, :n][fin] - exact[fin]).max() <= 1e-4 * cfg.layers * cfg.kv_heads
    pre = H.export_all(gpu, cfg)
    gpu.evict_global(12000)
    gpu.synchronize()
    gpu.poll_error()
    kept = O.select_keep(keys[0, :n], n, cfg.prompt, cfg.window, 12000)
    idx = torch.from_numpy(kept)
    assert gpu.len(0) == 12000 == len(kept)
    for key, (K0, V0, p0, s0) in pre.items():
        K1, V1, p1, s1 = gpu.export_slab(*key)
        assert torch.equal(p1, p0[idx]) and torch.equal(H.bits(s1), H.bits(s0[idx])), key
        assert torch.equal(H.bits(K1), H.bits(K0[idx])) and torch.equal(H.bits(V1), H.bits(V0[idx])), key
    gpu.close()
    torch.cuda.empty_cache()
