"""Pins for the oracle's method-level parts: the speculative cycle's invariants, the entropy
confidence (Eq. 1-4) and the adaptive-window selection (Eq. 5-10)."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import synth
from oracle.selection import SelectConfig, select_skip_set, selection_details

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    rows = {}
    plain = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        try:
            plain.append([float(p) for p in parts])
        except ValueError:
            rows[parts[0]] = [float(p) for p in parts[1:]]
    return rows, plain


# ---------------------------------------------------------------- cycle invariants

@pytest.fixture(scope="module")
def c1():
    w = synth.WORKLOADS["C1"]
    return w, synth.make_weights(w.shape, w.seed), synth.make_prompt(w.seed, w.prompt_len, w.shape.vocab)


def test_accept_greedy_definition():
    assert oracle.accept_greedy([5, 6, 7], [5, 6, 7, 8]) == (3, [5, 6, 7, 8])
    assert oracle.accept_greedy([5, 6, 7], [5, 9, 7, 8]) == (1, [5, 9])
    assert oracle.accept_greedy([5, 6, 7], [1, 6, 7, 8]) == (0, [1])
    assert oracle.accept_greedy([], [4]) == (0, [4])
    # a later match after a mismatch does not count (longest *prefix*)
    assert oracle.accept_greedy([1, 2, 3, 4], [1, 0, 3, 4, 5])[0] == 1


def test_empty_skip_set_accepts_everything(c1):
    w, W, p = c1
    for K in (1, 4, 7):
        s = oracle.generate_speculative(oracle.OracleModel(w.shape, W), p, None, K, 24)
        assert all(c["n_accepted"] == K for c in s["cycles"])
        assert s["alpha"] == 1.0 and s["M"] == K and s["beta"] == 0.0


@pytest.mark.parametrize("layers,K", [([1], 4), ([2], 4), ([1, 2], 4), ([1], 1), ([2], 7), ([0, 1, 2, 3], 3)])
def test_lossless_for_any_skip_set(c1, layers, K):
    """Speculative output equals vanilla greedy output token for token."""
    w, W, p = c1
    van = oracle.generate_vanilla(oracle.OracleModel(w.shape, W), p, w.gen_len)
    mask = synth.layers_to_mask(layers, w.shape.n_layers)
    s = oracle.generate_speculative(oracle.OracleModel(w.shape, W), p, mask, K, w.gen_len)
    assert s["tokens"] == van["tokens"]
    assert len(s["tokens"]) == w.gen_len
    emitted = 1 + sum(c["n_accepted"] + 1 for c in s["cycles"])
    assert emitted >= w.gen_len and emitted - (s["cycles"][-1]["n_accepted"] + 1) < w.gen_len
    assert s["alpha"] == s["accepted"] / (K * len(s["cycles"]))
    assert s["beta"] == len(layers) / w.shape.n_layers


def test_lossless_on_a_bf16_model():
    w = synth.reduced(synth.WORKLOADS["C2"], n_layers=4, prompt_len=12, gen_len=10)
    import dataclasses
    sh = dataclasses.replace(w.shape, vocab=512)
    W = synth.make_weights(sh, 5)
    p = synth.make_prompt(5, 12, sh.vocab)
    van = oracle.generate_vanilla(oracle.OracleModel(sh, W), p, 10)
    s = oracle.generate_speculative(oracle.OracleModel(sh, W), p, synth.layers_to_mask([1, 2], 4), 3, 10)
    assert s["tokens"] == van["tokens"]


# ---------------------------------------------------------------- confidence-aware drafting (early stop)

class _ScriptedModel:
    """Stands in for the transformer: the logits after a token are read from a table (one for the draft model, which
    is called with a skip mask, one for the target model), so every top-1 probability is known in closed form."""
    L = 4

    def __init__(self, draft_table, target_table):
        self.draft_table, self.target_table = draft_table, target_table

    def forward(self, tokens, pos, mask=None, want_hidden=False, want_logits=True):
        tab = self.target_table if mask is None else self.draft_table
        return {"logits": np.stack([np.asarray(tab[int(t)], np.float32) for t in tokens])}


def test_early_stop_on_a_scripted_model_with_known_probabilities():
    """Token 0 is followed by logits [0, 2, 1, 0] (greedy token 1, top-1 probability e^2 / (e^2 + e + 2) = 0.6103, the
    value of the confidence golden vector), token 1 by [0, 0, 1, 0] (greedy token 2, probability e / (e + 3) = 0.4754),
    token 2 by [0, 0, 0, 4] (token 3, e^4 / (e^4 + 3) = 0.9479), token 3 by [9, 0, 0, 0] (token 0, 0.9996)."""
    tab = {0: [0, 2, 1, 0], 1: [0, 0, 1, 0], 2: [0, 0, 0, 4], 3: [9, 0, 0, 0]}
    m = _ScriptedModel(tab, tab)
    mask = np.array([0, 3, 0, 0], np.uint8)
    c = oracle.speculative_cycle(m, mask, 0, 10, 4)                                  # no early stop: K drafts
    assert c["drafts"] == [1, 2, 3, 0] and c["n_drafted"] == 4 and c["n_accepted"] == 4
    assert c["draft_pmax"] == pytest.approx([0.610296, 0.475367, 0.947915, 0.999630], abs=2e-6)
    c = oracle.speculative_cycle(m, mask, 0, 10, 4, stop_p=0.5)                      # 0.61 >= 0.5 goes on, 0.4754 < 0.5 stops
    assert c["drafts"] == [1, 2] and c["n_drafted"] == 2
    assert c["targets"] == [1, 2, 3] and c["n_accepted"] == 2 and c["emitted"] == [1, 2, 3]   # the low-confidence draft is still verified
    c = oracle.speculative_cycle(m, mask, 0, 10, 4, stop_p=0.7)                      # already the first draft is below
    assert c["drafts"] == [1] and c["emitted"] == [1, 2] and c["new_ctx"] == 12
    c = oracle.speculative_cycle(m, mask, 0, 10, 4, stop_p=0.47)                     # 0.4754 >= 0.47: nothing stops
    assert c["n_drafted"] == 4
    c = oracle.speculative_cycle(m, mask, 2, 10, 3, stop_p=0.9999)                   # 0.9479 < 0.9999
    assert c["drafts"] == [3]
    # a target model that disagrees on the second token: the stop does not change what acceptance means
    tgt = dict(tab)
    tgt[1] = [0, 5, 0, 0]
    c = oracle.speculative_cycle(_ScriptedModel(tab, tgt), mask, 0, 10, 4, stop_p=0.5)
    assert c["drafts"] == [1, 2] and c["targets"][:2] == [1, 1] and c["n_accepted"] == 1 and c["emitted"] == [1, 1]


def test_early_stop_threshold_zero_is_fixed_k_and_counts_fall_with_the_threshold(c1):
    w, W, p = c1
    mask = synth.layers_to_mask([1], w.shape.n_layers)
    om = oracle.OracleModel(w.shape, W)
    t0 = oracle.prefill(om, p)[0]
    base = oracle.speculative_cycle(om, mask, t0, len(p), 6)
    zero = oracle.speculative_cycle(om, mask, t0, len(p), 6, stop_p=0.0)
    assert zero["drafts"] == base["drafts"] and zero["n_drafted"] == 6 and zero["emitted"] == base["emitted"]
    pm = base["draft_pmax"]
    assert all(0.0 < v <= 1.0 for v in pm)
    prev = 6
    for thr in sorted(set([0.0] + [v * (1 + 1e-9) for v in pm] + [v * (1 - 1e-9) for v in pm] + [1.0])):
        c = oracle.speculative_cycle(om, mask, t0, len(p), 6, stop_p=thr)
        # from the same state the drafts are a prefix of the fixed-K drafts, cut after the first one below the threshold
        want = next((i + 1 for i, v in enumerate(pm) if thr > 0 and v < thr), 6)
        assert c["n_drafted"] == want and c["drafts"] == base["drafts"][:want]
        assert c["n_drafted"] <= prev
        prev = c["n_drafted"]
    assert prev == 1                                                               # threshold 1.0 (above every probability here)


@pytest.mark.parametrize("stop_p", [0.002, 0.01, 1.0])
def test_early_stop_keeps_generation_lossless(c1, stop_p):
    w, W, p = c1
    van = oracle.generate_vanilla(oracle.OracleModel(w.shape, W), p, w.gen_len)
    s = oracle.generate_speculative(oracle.OracleModel(w.shape, W), p, synth.layers_to_mask([1, 2], w.shape.n_layers), 5,
                                    w.gen_len, stop_p=stop_p)
    assert s["tokens"] == van["tokens"]
    assert s["drafted"] == sum(c["n_drafted"] for c in s["cycles"]) <= 5 * len(s["cycles"])
    if stop_p == 1.0:
        assert all(c["n_drafted"] == 1 for c in s["cycles"])


# ---------------------------------------------------------------- confidence (Eq. 1-4)

def _brute(logits):
    l = np.asarray(logits, np.float64)
    p = np.exp(l - l.max()); p /= p.sum()
    H = -(p * np.log(p + 1e-10)).sum()
    return 1 - H / math.log(len(l)), p.max(), int(np.argmax(l))


def test_confidence_golden_check_vector():
    _, plain = _gold("confidence_check.txt")
    conf, pm, am = oracle.confidence_of_logits(np.array([2, 1, 0, 0], np.float32))
    assert abs(conf - plain[0][0]) < 5e-7 and abs(pm - plain[0][1]) < 5e-7 and am == int(plain[0][2])


def test_confidence_closed_forms():
    V = 1024
    conf, pm, am = oracle.confidence_of_logits(np.full(V, 3.25, np.float32))
    assert abs(conf) < 1e-6 and abs(pm - 1 / V) < 1e-12 and am == 0        # uniform -> 0, lowest index
    l = np.zeros(V, np.float32); l[77] = 80.0
    conf, pm, am = oracle.confidence_of_logits(l)
    assert abs(conf - 1) < 1e-9 and abs(pm - 1) < 1e-9 and am == 77         # one dominant logit -> 1
    l = np.full(V, -60.0, np.float32); l[3] = l[900] = 20.0
    conf, pm, am = oracle.confidence_of_logits(l)
    assert abs(conf - 0.9) < 1e-9 and abs(pm - 0.5) < 1e-9 and am == 3      # 1 - ln2/ln1024 = 0.9 exactly
    for v in (2, 7, 100):
        conf, _, _ = oracle.confidence_of_logits(np.random.default_rng(v).standard_normal(v).astype(np.float32))
        assert 0.0 <= conf <= 1.0


@pytest.mark.parametrize("V", [2, 5, 64, 1000, 1024])
def test_confidence_brute_force_and_invariances(V):
    rng = np.random.default_rng(V)
    l = (3 * rng.standard_normal(V)).astype(np.float32)
    conf, pm, am = oracle.confidence_of_logits(l)
    bc, bp, ba = _brute(l)
    assert abs(conf - bc) < 1e-12 and abs(pm - bp) < 1e-12 and am == ba
    conf2, pm2, am2 = oracle.confidence_of_logits((l.astype(np.float64) + 8.0).astype(np.float32))
    assert abs(conf2 - conf) < 1e-5 and abs(pm2 - pm) < 1e-5 and am2 == am  # shift invariance
    perm = rng.permutation(V)
    conf3, pm3, am3 = oracle.confidence_of_logits(l[perm])
    assert abs(conf3 - conf) < 1e-12 and abs(pm3 - pm) < 1e-12 and perm[am3] == am


def test_confidence_clamp_handles_huge_logits():
    l = np.zeros(16, np.float32); l[4] = np.inf; l[9] = -np.inf; l[2] = 3e38
    conf, pm, am = oracle.confidence_of_logits(l)
    assert np.isfinite(conf) and np.isfinite(pm)
    assert am == 2 and abs(pm - 0.5) < 1e-12                                  # both clamp to the same bound


def test_layer_confidences_permuting_head_rows():
    """Permuting LM-head rows permutes the greedy token and leaves confidence and p_max unchanged;
    c_layer is the plain mean over positions."""
    d, V = 64, 256
    g = torch.Generator().manual_seed(3)
    hidden = torch.randn(3, 5, d, generator=g).to(torch.bfloat16)
    head = (0.2 * torch.randn(V, d, generator=g)).to(torch.bfloat16)
    gain = 1.0 + 0.1 * torch.randn(d, generator=g)
    a = oracle.layer_confidences(hidden, head, gain)
    perm = torch.randperm(V, generator=g)
    b = oracle.layer_confidences(hidden, head[perm].contiguous(), gain)
    assert np.allclose(a["conf"], b["conf"], atol=1e-12) and np.allclose(a["p_max"], b["p_max"], atol=1e-12)
    assert np.array_equal(perm.numpy()[b["argmax"]], a["argmax"])
    assert np.allclose(a["c_layer"], a["conf"].mean(axis=1))
    # against a float64 torch evaluation of norm -> head -> softmax entropy
    h = hidden.double()
    r = h / torch.sqrt((h * h).mean(-1, keepdim=True) + 1e-5) * gain.double()
    lg = r @ head.double().T
    p = torch.softmax(lg, -1)
    conf = 1 + (p * torch.log(p + 1e-10)).sum(-1) / math.log(V)
    assert np.abs(a["conf"] - conf.numpy()).max() < 1e-6
    sub = oracle.layer_confidences(hidden, head, gain, rows=[2], positions=[1, 4])
    assert np.array_equal(sub["conf"], a["conf"][np.ix_([2], [1, 4])])


# ---------------------------------------------------------------- selection (Eq. 5-10)

def test_selection_golden_check_vector():
    rows, _ = _gold("selection_check.txt")
    c = [0.0] + rows["c"] + [0.0]
    cfg = SelectConfig(n_layers=12, lo=1, hi=10)
    d = selection_details(c, cfg)
    assert d["w_max"] == rows["w_max"][0]
    assert d["half"] == [int(v) for v in rows["half"]]
    assert np.abs(np.array(d["margin"]) - np.array(rows["margin"])).max() < 6e-5
    assert d["skip"] == [int(v) for v in rows["skip"]]
    assert select_skip_set(c, SelectConfig(n_layers=12, lo=1, hi=10, n_skip=3)) == [int(v) for v in rows["skip3"]]


def test_selection_constant_and_linear_profiles():
    L = 16
    cfg = SelectConfig(n_layers=L, n_skip=-1, min_ratio=0.0)
    d = selection_details([0.4] * L, cfg)
    assert d["skip"] == [] and all(m == 0 for m in d["margin"])               # constant -> nothing below its neighbours
    lin = [0.01 * i for i in range(L)]
    d = selection_details(lin, cfg)
    # a straight line has zero second difference everywhere (up to rounding noise, which the
    # epsilon of the min-max step keeps near 0), so w_i = w_base
    assert all(abs(w - cfg.w_base) < 1e-6 for w in d["w"])
    assert all(h == 1 for h in d["half"])
    # interior layers sit exactly on their neighbours' mean, so lambda*sigma > 0 keeps them
    assert not any(l in d["skip"] for l in d["layers"][2:-2])


def test_selection_single_dip_first_sorted_and_eligible_range():
    L = 20
    c = [0.5 + 0.01 * ((i * 7) % 5) for i in range(L)]
    c[9] = 0.05
    for n_skip in (1, 3, 6):
        S = select_skip_set(c, SelectConfig(n_layers=L, n_skip=n_skip))
        assert 9 in S and len(S) == n_skip and S == sorted(S)
        assert 0 not in S and L - 1 not in S                                     # first / last layer never eligible
    c2 = list(c); c2[0] = -5.0; c2[L - 1] = -5.0                                 # values outside the range are not read
    assert select_skip_set(c2, SelectConfig(n_layers=L, n_skip=3)) == select_skip_set(c, SelectConfig(n_layers=L, n_skip=3))
    S = select_skip_set(c, SelectConfig(n_layers=L, lo=4, hi=12, n_skip=4))
    assert all(4 <= l <= 12 for l in S)


def test_selection_minimum_ratio_and_lambda_monotone():
    rng = np.random.default_rng(4)
    L = 40
    c = list(0.3 + 0.1 * rng.standard_normal(L))
    base = selection_details(c, SelectConfig(n_layers=L, n_skip=-1, min_ratio=0.0))
    strict = [l for l, m in zip(base["layers"], base["margin"]) if m < 0]
    assert base["skip"] == strict                                                # Eq. 10, strict inequality
    S40 = select_skip_set(c, SelectConfig(n_layers=L, n_skip=-1, min_ratio=0.4))
    assert len(S40) >= int(math.floor(0.4 * 38 + 0.5)) and set(strict) <= set(S40) or len(strict) >= len(S40)
    sizes = [len(select_skip_set(c, SelectConfig(n_layers=L, lam=lam, n_skip=-1, min_ratio=0.0)))
             for lam in (0.0, 0.25, 0.5, 1.0, 2.0)]
    assert sizes == sorted(sizes, reverse=True)                                  # larger lambda -> fewer layers skipped
    # scale/shift of the confidences does not change the decision (Eq. 5 standardises)
    c3 = [3.0 * v + 1.0 for v in c]
    assert select_skip_set(c3, SelectConfig(n_layers=L, n_skip=10, flat_tol=0.0)) == \
        select_skip_set(c, SelectConfig(n_layers=L, n_skip=10, flat_tol=0.0))


def test_selection_window_grows_with_gradient_and_depth():
    L = 32
    c = [0.5] * L
    for i in range(1, 9):
        c[i] = 0.5                                                               # eight flat leading layers -> w_max = 8
    for i in range(9, L - 1):
        c[i] = 0.5 + (0.2 if i % 2 else -0.2) * (i / L)
    d = selection_details(c, SelectConfig(n_layers=L))
    assert d["w_max"] == 8.0
    w = d["w"]
    assert max(w) > 2.0 and w[0] == pytest.approx(2.0, abs=0.3)                  # Eq. 7: volatile deep layers get wider windows
    i_max = int(np.argmax(d["g"]))
    assert w[i_max] == pytest.approx(2.0 + 8.0 * 1.0 * (d["layers"][i_max] / L), rel=1e-6)
    fixed = selection_details(c, SelectConfig(n_layers=L, fixed_window=10))
    assert all(h == 5 for h in fixed["half"])


def test_score_loop_keeps_best_round_earliest_on_ties():
    cfg = SelectConfig(n_layers=10, n_skip=2)
    rng = np.random.default_rng(0)
    cs = [list(rng.random(10)) for _ in range(5)]
    out = oracle.score_loop(cs, [1.0, 3.0, 3.0, 2.0, 0.5], cfg)
    assert out["best_iter"] == 1 and out["best_set"] == select_skip_set(cs[1], cfg)
    assert len(out["sets"]) == 5


# ---------------------------------------------------------------- interval-based periodic search (Section 3.3)

def _search(c1, initial, K=3, max_new=60, interval=4, goal=10.0, max_rounds=3, P=8, taps=1):
    w, W, prompt = c1
    om = oracle.OracleModel(w.shape, W)
    cfg = SelectConfig(n_layers=w.shape.n_layers, lo=w.lo, hi=w.hi, n_skip=1)
    out = oracle.generate_search(om, W, prompt, initial, K, max_new, interval, goal, max_rounds, cfg, P, taps=taps)
    van = oracle.generate_vanilla(om, prompt, max_new)
    om.close()
    return out, van


def test_search_is_lossless_halts_and_keeps_the_best_round(c1):
    out, van = _search(c1, [1, 2])
    assert out["tokens"] == van["tokens"]                              # the search never changes the output
    assert 1 <= len(out["scores"]) <= 3 + 1 and not out["searching"]   # initial set + at most max_rounds searched sets
    best = int(np.argmax(out["scores"]))                               # first maximum: ties keep the earlier set
    assert out["best_round"] == best and out["best_set"] == out["sets"][best]
    assert out["final_set"] == out["best_set"]
    assert all(0.0 <= s <= 3.0 for s in out["scores"])                 # mean accepted per cycle lies in [0, K]
    for s in out["sets"][1:]:
        assert len(s) == 1 and s[0] in (1, 2)                          # searched sets come from the selection rule


def test_search_goal_and_interval_edges(c1):
    out, _ = _search(c1, [2], goal=0.0)                                # any score reaches a goal of 0: round 0 ends it
    assert len(out["scores"]) == 1 and out["final_set"] == [2] and not out["searching"]
    out, _ = _search(c1, [], K=3, goal=3.0)                            # empty skip set: every draft accepted, score = K
    assert out["scores"] == [3.0] and out["final_set"] == []
    out, _ = _search(c1, [1], interval=1000)                           # the interval never completes: no search check
    assert out["scores"] == [] and out["searching"] and out["final_set"] == [1]
    out, van = _search(c1, [1, 2], taps=2)                             # two taps per layer: still lossless, still halts
    assert out["tokens"] == van["tokens"] and not out["searching"]
    out, _ = _search(c1, [1], max_rounds=0)                            # no searched set allowed: only the initial one is scored
    assert len(out["scores"]) == 1 and out["final_set"] == [1]
