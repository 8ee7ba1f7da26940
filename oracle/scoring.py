"""All-layer early-exit confidence scoring and the search-round loop -- test infrastructure only.

Section 3.1: every layer's hidden state is projected through the (final norm and) shared LM head,
the logits are cast to FP32 and clamped, and the confidence is 1 - H(softmax) / log V (Eq. 1-4).
A layer's confidence is the arithmetic mean over the scored positions of the context window.
Section 3.3 / Appendix D: search rounds score, select a skip set (Eq. 5-10) and keep the best set.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List, Optional, Sequence

import numpy as np

from .model import CLAMP, EPS_H, _as_host_array, _ptr, lib
from .selection import SelectConfig, select_skip_set


def _to_f32(hidden) -> np.ndarray:
    if isinstance(hidden, np.ndarray):
        return np.ascontiguousarray(hidden, dtype=np.float32)
    return hidden.detach().cpu().float().contiguous().numpy()


def layer_confidences(hidden, lm_head, final_norm, rms_eps: float = 1e-5,
                      rows: Optional[Sequence[int]] = None, positions: Optional[Sequence[int]] = None
                      ) -> Dict[str, np.ndarray]:
    """hidden [R, P, d] (bf16 tensor or fp32 array); lm_head [V, d] (bf16 / fp16 tensor or fp32); final_norm fp32 [d].

    Returns conf, p_max (float64 [R', P']), argmax (int32), margin (top-2 logit gap) and
    c_layer (float64 [R'] = mean of conf over positions), restricted to the requested rows /
    positions (all by default).
    """
    h = _to_f32(hidden)
    R, P, d = h.shape
    W = _as_host_array(lm_head)
    wd = 1 if W.dtype == np.uint16 else 2 if W.dtype == np.float16 else 0
    V = W.shape[0]
    g = np.ascontiguousarray(_to_f32(final_norm))
    rows = list(range(R)) if rows is None else list(rows)
    positions = list(range(P)) if positions is None else list(positions)
    sel = np.ascontiguousarray(h[np.ix_(rows, positions)].reshape(-1, d))
    n = sel.shape[0]
    normed = np.empty_like(sel)
    for i in range(n):
        lib().orc_rmsnorm(_ptr(sel[i]), _ptr(g), d, rms_eps, _ptr(normed[i]))
    conf = np.empty(n, np.float64)
    pmax = np.empty(n, np.float64)
    amax = np.empty(n, np.int32)
    marg = np.empty(n, np.float64)
    chunk = 64
    logits = np.empty((chunk, V), np.float32)
    cf, pm, am = C.c_double(), C.c_double(), C.c_int()
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        lib().orc_matmul_rows(_ptr(W), wd, V, d, _ptr(normed[s:s + m]), m, _ptr(logits))
        for i in range(m):
            row = logits[i]
            lib().orc_confidence(_ptr(row), V, CLAMP, EPS_H, C.byref(cf), C.byref(pm), C.byref(am))
            conf[s + i], pmax[s + i], amax[s + i] = cf.value, pm.value, am.value
            part = np.partition(row.astype(np.float64), -2)
            marg[s + i] = part[-1] - part[-2]
    shp = (len(rows), len(positions))
    conf = conf.reshape(shp)
    return dict(conf=conf, p_max=pmax.reshape(shp), argmax=amax.reshape(shp), margin=marg.reshape(shp),
                c_layer=conf.mean(axis=1))


def score_loop(c_layers: Sequence[Sequence[float]], scores: Sequence[float], cfg: SelectConfig) -> Dict[str, object]:
    """Search rounds (Section 3.3, Appendix D): round t selects a skip set from that round's layer
    confidences; the set of the round with the highest score is kept (earliest round wins ties)."""
    sets: List[List[int]] = [select_skip_set(c, cfg) for c in c_layers]
    best = 0
    for t in range(1, len(sets)):
        if float(scores[t]) > float(scores[best]):
            best = t
    return dict(sets=sets, best_iter=best, best_set=sets[best] if sets else [])
