"""Draft / verify / greedy-accept cycle of self-speculative decoding (test infrastructure only).

Follows the generation step of Section 3 (Figure 2): the draft model -- the target model without
the layers of the skip set S -- proposes K candidate tokens one by one; the target model checks
them in a single forward pass; the longest prefix of candidates that equals the target's own
greedy choices is kept, plus one token from the target (lossless under greedy decoding,
Section 1 and Section 4.2).

One KV cache serves both models: the draft pass writes entries of kept layers only, the verify
pass rewrites every layer's entries for the positions it covers, and rejected positions are
simply overwritten by the next cycle (the cache length is a counter).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np


def top2_margin(logits_row: np.ndarray) -> float:
    """top-1 minus top-2 logit (how safely the greedy choice is decided)."""
    if logits_row.shape[0] < 2:
        return float("inf")
    part = np.partition(logits_row.astype(np.float64), -2)
    return float(part[-1] - part[-2])


def greedy_token(logits_row: np.ndarray) -> int:
    """argmax with the lowest index among equal maxima."""
    return int(np.argmax(logits_row))


def accept_greedy(drafts: Sequence[int], targets: Sequence[int]):
    """drafts d_1..d_K, targets g_1..g_{K+1} (g_i = target's greedy token after row i-1).
    n = largest i with d_j = g_j for all j <= i; emitted = d_1..d_n, g_{n+1}."""
    n = 0
    while n < len(drafts) and int(drafts[n]) == int(targets[n]):
        n += 1
    return n, [int(t) for t in drafts[:n]] + [int(targets[n])]


def top1_probability(logits_row: np.ndarray) -> float:
    """max of softmax(logits) in double (the draft's own confidence in its greedy token)."""
    l = logits_row.astype(np.float64)
    e = np.exp(l - l.max())
    return float(e.max() / e.sum())


def speculative_cycle(model, skip_mask: Optional[np.ndarray], t0: int, ctx: int, K: int,
                      want_hidden: bool = False, stop_p: float = 0.0) -> Dict[str, object]:
    """One cycle from the state (cache valid for positions < ctx, pending token t0).

    stop_p > 0 is the confidence-aware drafting the paper takes over from SWIFT (Section 3): drafting ends after
    the first candidate whose top-1 probability under the draft model is below stop_p.  That candidate is still
    handed to the target model (reading: the paper gives neither the threshold nor which side of it the last
    candidate falls on); stop_p = 0 always drafts K candidates."""
    drafts: List[int] = []
    d_margin: List[float] = []
    d_logits: List[np.ndarray] = []
    d_pmax: List[float] = []
    tok = int(t0)
    for i in range(K):
        lg = model.forward([tok], ctx + i, skip_mask)["logits"][0]
        tok = greedy_token(lg)
        drafts.append(tok)
        d_margin.append(top2_margin(lg))
        d_logits.append(lg)
        d_pmax.append(top1_probability(lg))
        if stop_p > 0.0 and d_pmax[-1] < stop_p:
            break
    nd = len(drafts)
    rows = [int(t0)] + drafts
    ver = model.forward(rows, ctx, None, want_hidden=want_hidden)
    vlog = ver["logits"]
    targets = [greedy_token(vlog[i]) for i in range(nd + 1)]
    v_margin = [top2_margin(vlog[i]) for i in range(nd + 1)]
    n, emitted = accept_greedy(drafts, targets)
    return dict(drafts=drafts, targets=targets, n_accepted=n, emitted=emitted, draft_margins=d_margin,
                verify_margins=v_margin, draft_logits=d_logits, verify_logits=vlog, draft_pmax=d_pmax, n_drafted=nd,
                hid_attn=ver.get("hid_attn"), hid_ffn=ver.get("hid_ffn"), new_ctx=ctx + n + 1, next_t0=emitted[-1])


def prefill(model, prompt: Sequence[int], want_hidden: bool = False):
    """Full model over the prompt from an empty cache; returns (first token, its margin, forward dict)."""
    out = model.forward(np.asarray(prompt, np.int32), 0, None, want_hidden=want_hidden)
    last = out["logits"][-1]
    return greedy_token(last), top2_margin(last), out


def generate_vanilla(model, prompt: Sequence[int], max_new: int) -> Dict[str, object]:
    """Plain autoregressive greedy decoding with the full model: the lossless reference."""
    t0, m0, _ = prefill(model, prompt)
    out, margins = [t0], [m0]
    ctx = len(prompt)
    while len(out) < max_new:
        lg = model.forward([out[-1]], ctx, None)["logits"][0]
        out.append(greedy_token(lg))
        margins.append(top2_margin(lg))
        ctx += 1
    return dict(tokens=out[:max_new], margins=margins[:max_new])


def generate_speculative(model, prompt: Sequence[int], skip_mask: Optional[np.ndarray], K: int,
                         max_new: int, stop_p: float = 0.0) -> Dict[str, object]:
    """Self-speculative greedy decoding: prefill, then cycles until max_new tokens are emitted
    (the last cycle's emission is truncated).  Statistics as defined in Section 4.1.2:
    alpha = accepted / drafted, M = mean accepted per cycle, beta = |S| / L."""
    t0, m0, _ = prefill(model, prompt)
    out = [t0]
    ctx = len(prompt)
    cycles: List[Dict[str, object]] = []
    while len(out) < max_new:
        cyc = speculative_cycle(model, skip_mask, out[-1], ctx, K, stop_p=stop_p)
        cyc["ctx"] = ctx
        cyc["t0"] = out[-1]
        cycles.append(cyc)
        out.extend(cyc["emitted"])
        ctx = cyc["new_ctx"]
    drafted = sum(c["n_drafted"] for c in cycles)
    accepted = sum(c["n_accepted"] for c in cycles)
    L = model.L
    n_skipped = 0 if skip_mask is None else int(np.count_nonzero(np.asarray(skip_mask)))
    return dict(tokens=out[:max_new], first_margin=m0, cycles=cycles, drafted=drafted, accepted=accepted,
                alpha=(accepted / drafted if drafted else 0.0),
                M=(accepted / len(cycles) if cycles else 0.0), beta=n_skipped / L)
