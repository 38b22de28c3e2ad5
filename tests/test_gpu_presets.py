"""The comparison tables' structural policies (Table 1: Window, StreamingLLM-shaped; Table 2:
T-Random, T-Bottom, without the question window, without the local window) are parameterisations of
the same decode / append-score / select-at-budget calls.  Each preset runs a whole trajectory on
the device and must equal the oracle driven with the same parameters written out here by hand:
retained positions, K, V and scores bit for bit, lengths equal to Section 5's closed form, and
the property that names the policy (what the retained set consists of)."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O
from tests import helpers as H

# name -> (question rows pinned, local window, ratio, sign/kind of the appended score)
B, M, WL, R, SINKS, STEPS = 128, 24, 16, 0.25, 4, 260
TABLE = {
    "dynts": (M, WL, R, "pred"),
    "attention": (M, WL, R, None),
    "window": (0, WL, 0.0, "zero"),
    "streaming": (SINKS, WL, 0.0, "zero"),
    "t_random": (M, WL, R, "rand"),
    "t_bottom": (M, WL, R, "neg"),
    "wo_q": (0, WL, R, "pred"),
    "wo_l": (M, 0, R, "pred"),
}


def _pred(s, batch):
    return np.random.default_rng([5, s]).standard_normal(batch).astype(np.float32)


def _rand(s, batch):
    return np.random.default_rng([6, s]).random(batch, dtype=np.float32)


def test_preset_table_and_closed_form_lengths():
    """Host logic only: the presets carry the parameters of the table above and their length curve
    is the oracle's S_i = M + i - n_i K."""
    from paper_2601_18383_b200 import presets as P
    assert set(P.NAMES) == set(TABLE)
    for name, (pin, wl, r, kind) in TABLE.items():
        p = P.make(name, B, WL, R, M, sinks=SINKS)
        assert (p.n_pinned, p.window, p.ratio) == (pin, wl, r), name
        keep = O.paper_target(pin, B, wl, r)
        assert p.kept_after_event() == keep and p.evicted_per_event() == B - keep
        assert p.lengths(M, STEPS) == [O.effective_length(M, i, B, B - keep) for i in range(1, STEPS + 1)]
    with pytest.raises(ValueError):
        P.make("dynts", B, WL, 1.0, M)          # keeps everything: never evicts
    with pytest.raises(ValueError):
        P.make("dynts", 32, 16, 0.5, 24)        # no selection window
    with pytest.raises(ValueError):
        P.make("h2o", B, WL, R, M)


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(TABLE))
def test_preset_trajectory_equals_oracle(name):
    import paper_2601_18383_b200 as D
    from paper_2601_18383_b200 import presets as P
    pin, wl, r, kind = TABLE[name]
    cfg = W.get_config("c2_llama8b").scaled(layers=2, batch=2, prompt=M, budget=B, window=wl, evict_interval=1)
    preset = P.make(name, B, WL, R, M, sinks=SINKS)
    run = P.PresetRun(preset, cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim, dtype=cfg.dtype)
    gpu = run.cache
    orc = H.make_oracle(cfg)
    pk, pv = W.prompt_kv(cfg, 31)
    run.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    O.prefill(orc, pk.astype(np.float64), pv.astype(np.float64), n_pinned=pin)
    stream = W.DecodeStream(cfg, 31)
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=H.tdtype(cfg), device="cuda:0")
    keep = O.paper_target(pin, B, wl, r)
    pred_of_pos = {}                                  # position -> predictor score, per sequence 0
    events = 0
    for s in range(1, STEPS + 1):
        q, k, v = stream.step(s)
        pr, rn = _pred(s, cfg.batch), _rand(s, cfg.batch)
        pred_of_pos[M + s - 1] = float(pr[0])
        O.decode_step(orc, q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), accumulate=kind is None)
        if kind is None and orc.length(0) >= B:
            # accumulated mass is fp32 on the device and float64 in the oracle: the selection is an
            # integer decision, so both sides take it from the same (the device's) score values
            gpu.decode_attn(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out)
            for l, b, h, sl in orc.units():
                sc = gpu.export_slab(l, b, h)[3].numpy().astype(np.float64)
                assert np.abs(sc[pin:] - sl.score[pin:sl.n]).max() <= H.TOL_DELTA * 4
                sl.score[:sl.n] = sc
            before = gpu.len(0)
            gpu.evict_at_budget(B, r)
            run.events += int(gpu.len(0) < before)
        else:
            run.step(H.dev(q, cfg), H.dev(k, cfg), H.dev(v, cfg), out, torch.from_numpy(pr).cuda(), torch.from_numpy(rn).cuda())
        if kind is not None:
            O.set_new_scores(orc, {"pred": pr, "neg": -pr, "rand": rn, "zero": np.zeros_like(pr)}[kind])
        fired = orc.length(0) >= B
        if fired:
            O.evict(orc, keep)
            events += 1
        assert gpu.len(0) == orc.length(0) == preset.length_after(M, s), (name, s)
        if fired or s == STEPS:
            for l, b, h, sl in orc.units():
                Kd, Vd, pos, score = gpu.export_slab(l, b, h)
                assert np.array_equal(pos.numpy(), sl.pos[:sl.n]), (name, s, l, b, h)
                assert np.array_equal(Kd.to(torch.float64).numpy(), sl.K[:sl.n])
                assert np.array_equal(Vd.to(torch.float64).numpy(), sl.V[:sl.n])
                if kind is not None or fired:
                    assert np.array_equal(score.numpy().astype(np.float64), sl.score[:sl.n])
        if fired:                                   # the property that names the policy, sequence 0, slab (0, 0, 0)
            pos = gpu.export_slab(0, 0, 0)[2].numpy()
            newest = M + s - 1
            recent = set(range(newest - wl + 1, newest + 1))
            if name == "window":
                assert set(pos) == recent
            elif name == "streaming":
                assert set(pos) == set(range(SINKS)) | recent
            else:
                assert set(range(pin)) <= set(pos) and recent <= set(pos)
            if name in ("dynts", "t_bottom") and events == 1:
                # first event: every candidate still carries its own predictor score
                cand = [p_ for p_ in range(M, newest - wl + 1)]
                order = sorted(cand, key=lambda p_: (-pred_of_pos[p_], p_) if name == "dynts" else (pred_of_pos[p_], p_))
                chosen = set(order[: keep - pin - wl])
                assert set(pos) - set(range(pin)) - recent == chosen
    assert events == run.events and events >= 2
    gpu.poll_error()
    run.close()
