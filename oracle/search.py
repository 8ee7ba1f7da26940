"""Generation with the interval-based periodic search (Section 3.3, Figure 2) -- test infrastructure only.

The current skip set serves as the draft model for `interval` draft/verify/accept cycles (Opt_Interval) while the
number of accepted candidates is accumulated.  At the end of an interval the search check computes the round's
score (mean accepted candidates per cycle); the best-scoring set so far is kept; the search stops once a score
reaches the goal or the maximum number of search rounds has been evaluated, and the best saved set then drafts
for the rest of the generation.  Otherwise the layer confidences (Section 3.1) of the hidden states in the
context window are computed, a new skip set is selected (Section 3.2) and installed, and a new interval starts.

Readings (the paper leaves them open): the initial, uniformly skipped set is round 0 and is scored like the
others; `max_rounds` counts the searched sets after it; the context window is a ring of the last P positions of
the verify passes (slot = position mod P), filled by the prefill and by every verify pass while the search is
on, rejected rows included until a later pass overwrites them; the score is accepted / interval; ties keep the
earlier set.  The output tokens never depend on any of this (greedy acceptance is lossless).
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from .cycle import prefill, speculative_cycle
from .scoring import layer_confidences
from .selection import SelectConfig, select_skip_set


def _mask_of(layers: Sequence[int], n_layers: int) -> np.ndarray:
    m = np.zeros(n_layers, np.uint8)
    for l in layers:
        m[int(l)] = 3
    return m


def generate_search(model, weights: Dict[str, object], prompt: Sequence[int], initial_set: Sequence[int], K: int,
                    max_new: int, interval: int, score_goal: float, max_rounds: int, select_cfg: SelectConfig,
                    P: int, storage_dtype=None, taps: int = 1) -> Dict[str, object]:
    """Returns tokens (max_new of them, the first being the prefill's), per-round scores and sets, the best round
    and the set in use at the end.  `weights` supplies lm_head and final_norm for the confidence scoring;
    `storage_dtype` (a torch dtype or None) is the type the ring rounds hidden states to.  taps = 2 also records the
    stream after each layer's attention add (Section 3.1 names both modules); a layer's confidence is then the mean
    over both taps and all positions."""
    import torch
    L, d = model.L, model.d
    t0, _, pre = prefill(model, prompt, want_hidden=True)
    ring = np.zeros((L, taps, P, d), np.float32)

    def store(fwd, pos0):   # fwd: forward dict with hid_attn / hid_ffn [L, n, d]: rows at positions pos0 ..
        for ti, key in enumerate(("hid_attn", "hid_ffn") if taps == 2 else ("hid_ffn",)):
            h = torch.tensor(fwd[key])
            if storage_dtype is not None:
                h = h.to(storage_dtype).float()
            for i in range(h.shape[1]):
                ring[:, ti, (pos0 + i) % P, :] = h[:, i, :].numpy()

    store(pre, 0)
    out = [t0]
    ctx = len(prompt)
    cur = sorted(int(l) for l in initial_set)
    sets: List[List[int]] = []
    scores: List[float] = []
    best_set, best_score, best_round = list(cur), -np.inf, 0
    searching, rnd = True, 0
    it, acc = 0, 0
    while len(out) < max_new:
        cyc = speculative_cycle(model, _mask_of(cur, L), out[-1], ctx, K, want_hidden=searching)
        if searching:
            store(cyc, ctx)
        out.extend(cyc["emitted"])
        ctx = cyc["new_ctx"]
        if not searching:
            continue
        it += 1
        acc += cyc["n_accepted"]
        if it < interval:
            continue
        score = acc / float(interval)          # search check at the end of the interval
        sets.append(list(cur))
        scores.append(score)
        if score > best_score:
            best_set, best_score, best_round = list(cur), score, rnd
        if score >= score_goal or rnd >= max_rounds:
            searching = False
            cur = list(best_set)
        else:
            h = torch.tensor(ring.reshape(L, taps * P, d))
            if storage_dtype is not None:
                h = h.to(storage_dtype)
            c = layer_confidences(h, weights["lm_head"], weights["final_norm"], model.shape.rms_eps)["c_layer"]
            cur = select_skip_set([float(np.float32(v)) for v in c], select_cfg)
            rnd += 1
        it, acc = 0, 0
    return dict(tokens=out[:max_new], scores=scores, sets=sets, best_round=best_round, best_set=best_set,
                final_set=cur, searching=searching)
