"""Selection policies of the paper's comparison tables as parameterisations of the same calls.

Every row below runs the SAME kernels: the fused decode step, `dynts_append_scores` and
`dynts_evict_at_budget`.  What differs is host-side only -- how many prompt rows are pinned (the
question window W_q), the local window W_l, the retention ratio r of the selection window W_s, and
which number is appended as the new token's score:

  dynts       Section 4.2: question pinned, local window kept, top r W_s by the predictor's score
  attention   the same layout with accumulated attention mass (Eq. 6) as the score; nothing appended
  window      "Window" of Table 1: only the most recent tokens survive (no pins, r = 0)
  streaming   StreamingLLM-shaped: a few sink rows pinned + the local window, r = 0
  t_random    Table 2: the retained thinking tokens are chosen at random (uniform scores)
  t_bottom    Table 2: the LOWEST-scored thinking tokens are retained (negated scores)
  wo_q        Table 2, without the question: the prompt rows compete like any other row
  wo_l        Table 2, without the local window: W_l = 0

No arithmetic of the method lives here: the module only chooses arguments.  Random numbers are the
caller's (passed to `step_scores`), so a run is reproducible from its seeds.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

from . import binding as _b

NAMES = ("dynts", "attention", "window", "streaming", "t_random", "t_bottom", "wo_q", "wo_l")


@dataclass(frozen=True)
class Preset:
    name: str
    budget: int            # B: the row count that triggers a selection
    window: int            # W_l given to the cache
    ratio: float           # r: share of the selection window that survives
    n_pinned: int          # W_q: prompt rows that are never evicted
    score_source: int      # DYNTS_SCORE_ATTENTION or DYNTS_SCORE_EXTERNAL
    score_kind: str        # "predictor", "negated", "random", "zero", "none"

    def step_scores(self, predictor_scores, random_scores=None):
        """The tensor to append after a decode step (None: nothing is appended)."""
        if self.score_kind == "none":
            return None
        if self.score_kind == "predictor":
            return predictor_scores
        if self.score_kind == "negated":
            return -predictor_scores
        if self.score_kind == "random":
            if random_scores is None:
                raise ValueError("t_random needs the caller's random numbers")
            return random_scores
        return predictor_scores * 0

    def kept_after_event(self) -> int:
        """Rows left by a selection: W_q + floor(r W_s) + W_l with W_s = B - W_q - W_l."""
        ws = self.budget - self.n_pinned - self.window
        return self.n_pinned + int(math.floor(self.ratio * ws)) + self.window

    def evicted_per_event(self) -> int:
        return self.budget - self.kept_after_event()

    def length_after(self, prompt: int, steps: int) -> int:
        """Rows held after `steps` decode steps from a prompt of `prompt` rows (Section 5: the
        length grows by one per step and drops by K each time it reaches B)."""
        n, K = prompt + steps, self.evicted_per_event()
        if n < self.budget or K <= 0:
            return n
        return n - ((n - self.budget) // K + 1) * K

    def lengths(self, prompt: int, steps: int) -> List[int]:
        return [self.length_after(prompt, s) for s in range(1, steps + 1)]


def make(name: str, budget: int, window: int, ratio: float, prompt: int, sinks: int = 4) -> Preset:
    """`prompt` = rows of the question; `sinks` = pinned rows of the streaming preset."""
    ext, att = _b.DYNTS_SCORE_EXTERNAL, _b.DYNTS_SCORE_ATTENTION
    if name == "dynts":
        p = Preset(name, budget, window, ratio, prompt, ext, "predictor")
    elif name == "attention":
        p = Preset(name, budget, window, ratio, prompt, att, "none")
    elif name == "window":
        p = Preset(name, budget, window, 0.0, 0, ext, "zero")
    elif name == "streaming":
        p = Preset(name, budget, window, 0.0, min(sinks, prompt), ext, "zero")
    elif name == "t_random":
        p = Preset(name, budget, window, ratio, prompt, ext, "random")
    elif name == "t_bottom":
        p = Preset(name, budget, window, ratio, prompt, ext, "negated")
    elif name == "wo_q":
        p = Preset(name, budget, window, ratio, 0, ext, "predictor")
    elif name == "wo_l":
        p = Preset(name, budget, 0, ratio, prompt, ext, "predictor")
    else:
        raise ValueError(f"unknown preset {name!r}; one of {NAMES}")
    if p.n_pinned + p.window >= p.budget:
        raise ValueError("W_q + W_l must leave a selection window below the budget")
    if p.evicted_per_event() <= 0:
        raise ValueError("the ratio keeps the whole selection window: nothing would be evicted")
    return p


class PresetRun:
    """A cache driven by a preset: prefill, then `step` per generated token."""

    def __init__(self, preset: Preset, layers, batch, q_heads, kv_heads, head_dim, dtype="bf16", device="cuda:0"):
        self.preset = preset
        # One spare row is enough for the trigger-at-B schedule; the row count of a slab is rounded up
        # to a multiple of 32 so that the kernels' vector paths apply (16-byte score accesses, whole
        # 128-byte lines of the logit scratch).
        capacity = (preset.budget + 1 + 31) // 32 * 32
        self.cache = _b.Cache(layers, batch, q_heads, kv_heads, head_dim, preset.budget, preset.window, 1,
                              dtype=dtype, capacity=capacity, device=device)
        self.cache.set_score_source(preset.score_source)
        self.events = 0

    def prefill(self, k, v, q=None, out=None):
        if q is not None:
            self.cache.prefill_attn(q, k, v, out, n_pinned=self.preset.n_pinned)
        else:
            self.cache.prefill(k, v, n_pinned=self.preset.n_pinned)

    def step(self, q, k_new, v_new, out, predictor_scores=None, random_scores=None, delta: Optional[object] = None):
        c, p = self.cache, self.preset
        c.decode_attn(q, k_new, v_new, out, delta)
        s = p.step_scores(predictor_scores, random_scores)
        if s is not None:
            c.append_scores(s)
        before = c.len(0)
        c.evict_at_budget(p.budget, p.ratio)
        if c.len(0) < before:
            self.events += 1

    def close(self):
        self.cache.close()
