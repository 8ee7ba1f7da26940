"""Adaptive confidence-window skip-set selection (Section 3.2, Eq. 5-10) -- test infrastructure only.

Plain Python floats (IEEE double), one scalar operation per line of the definitions, so that it
can be read against the equations.  Where the paper leaves a detail open the reading taken is
stated at the step that needs it.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Sequence


@dataclasses.dataclass
class SelectConfig:
    n_layers: int                 # total layers of the model (num_layers in Eq. 7)
    lo: int = 1                   # first eligible layer (first and last layer are never considered, App. B)
    hi: int = -1                  # last eligible layer, inclusive (-1: n_layers - 2)
    w_base: float = 2.0           # Section 4.1.1
    lam: float = 0.3              # threshold sensitivity, 0.25 < lambda < 0.5 (Section 4.1.1)
    eps: float = 1e-8             # epsilon of Eq. 5 and of the min-max rescaling
    flat_tol: float = 1e-3        # "same confidence value" tolerance for w_max
    w_max: float = 0.0            # <= 0: count of leading eligible layers sharing the first value
    n_skip: int = -1              # >= 0: exactly this many layers; < 0: Eq. 10 plus the minimum ratio
    min_ratio: float = 0.4        # minimum skip ratio (Section 4.1.1)
    fixed_window: int = 0         # > 0: constant window (ablation of Section 4.3.2) instead of Eq. 7

    def __post_init__(self):
        if self.hi < 0:
            self.hi = self.n_layers - 2


def _gradient(x: Sequence[float]) -> List[float]:
    """First-order discrete gradient: central differences inside, one-sided at the two ends."""
    n = len(x)
    if n < 2:
        return [0.0] * n
    out = [0.0] * n
    out[0] = x[1] - x[0]
    out[n - 1] = x[n - 1] - x[n - 2]
    for i in range(1, n - 1):
        out[i] = (x[i + 1] - x[i - 1]) * 0.5
    return out


def selection_details(c_layer: Sequence[float], cfg: SelectConfig) -> Dict[str, object]:
    """All intermediate quantities of Eq. 5-10 for the eligible layers lo..hi.

    c_layer is indexed by model layer (length n_layers); only entries lo..hi are read.
    """
    lo, hi, L = cfg.lo, cfg.hi, cfg.n_layers
    n = hi - lo + 1
    if n <= 0:
        return dict(layers=[], chat=[], g=[], w=[], half=[], margin=[], skip=[], w_max=0.0)
    c = [float(c_layer[lo + i]) for i in range(n)]

    # Eq. 5: standardise over the eligible layers (population standard deviation).
    s = 0.0
    for v in c:
        s += v
    mu = s / n
    s = 0.0
    for v in c:
        s += (v - mu) * (v - mu)
    sigma = math.sqrt(s / n)
    chat = [(v - mu) / (sigma + cfg.eps) for v in c]

    # Eq. 6: second-order discrete gradient = the gradient operator applied twice; its magnitude,
    # min-max rescaled to [0, 1].  Fewer than three layers have no second difference: g = 0.
    if n >= 3:
        g = [abs(v) for v in _gradient(_gradient(chat))]
    else:
        g = [0.0] * n
    gmin, gmax = min(g), max(g)
    g = [(v - gmin) / (gmax - gmin + cfg.eps) for v in g]

    # w_max: number of leading eligible layers whose confidence equals the first one's
    # (within flat_tol) before any change occurs.
    if cfg.w_max > 0:
        w_max = float(cfg.w_max)
    else:
        cnt = 0
        for v in c:
            if abs(v - c[0]) <= cfg.flat_tol:
                cnt += 1
            else:
                break
        w_max = float(max(cnt, 1))

    # Eq. 7: w_i = w_base + w_max * g_i * (l_i / num_layers), l_i the 0-based model layer index.
    w = [cfg.w_base + (w_max * g[i]) * ((lo + i) / L) for i in range(n)]

    # Window as a set: W_i = round-half-up(w_i) neighbours in total, split on both sides,
    # current layer excluded, clipped to the eligible range.
    half = []
    for i in range(n):
        W = cfg.fixed_window if cfg.fixed_window > 0 else int(math.floor(w[i] + 0.5))
        half.append(max(1, (W + 1) // 2))

    # Eq. 8-10: local mean / population std over the window, margin = c_hat - (mu - lambda sigma).
    margin, mu_loc, sd_loc = [], [], []
    for i in range(n):
        a, b = max(0, i - half[i]), min(n - 1, i + half[i])
        s, cnt = 0.0, 0
        for j in range(a, b + 1):
            if j != i:
                s += chat[j]
                cnt += 1
        if cnt == 0:
            m_i, sd_i = chat[i], 0.0
        else:
            m_i = s / cnt
            s = 0.0
            for j in range(a, b + 1):
                if j != i:
                    s += (chat[j] - m_i) * (chat[j] - m_i)
            sd_i = math.sqrt(s / cnt)
        mu_loc.append(m_i)
        sd_loc.append(sd_i)
        margin.append(chat[i] - (m_i - cfg.lam * sd_i))

    # Eq. 10 (strict) and the skip-ratio post-step.
    order = sorted(range(n), key=lambda i: (margin[i], i))      # smallest margin first, ties -> lower layer
    if cfg.n_skip >= 0:
        chosen = set(order[: min(cfg.n_skip, n)])
    else:
        chosen = {i for i in range(n) if margin[i] < 0.0}
        need = int(math.floor(cfg.min_ratio * n + 0.5))
        for i in order:
            if len(chosen) >= need:
                break
            chosen.add(i)
    skip = sorted(lo + i for i in chosen)                        # sorted by index (end of Section 3.2)
    return dict(layers=[lo + i for i in range(n)], chat=chat, g=g, w=w, half=half, mu_local=mu_loc,
                sd_local=sd_loc, margin=margin, skip=skip, w_max=w_max)


def select_skip_set(c_layer: Sequence[float], cfg: SelectConfig) -> List[int]:
    """Sorted list of layers to skip."""
    return selection_details(c_layer, cfg)["skip"]
