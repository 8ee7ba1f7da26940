"""Run-time behaviour of the library on a B200 that is not a numerical comparison: the bounded-wait path, error
flags, argument ranges and bit reproducibility.  Nothing here faults, traps or hangs the GPU: the one wait that is
made to run out is a grid barrier that is told to expect one arrival more than there are CTAs, with a bound of a
few milliseconds, after which the kernel returns by itself."""
import dataclasses

import numpy as np
import pytest

import oracle
import paper_2604_14612_b200 as cl
import synth
from paper_2604_14612_b200.binding import CL_DEBUG_BARRIER_EXTRA, CL_DEBUG_DEVICE_ERR, CL_DEBUG_WAIT_LIMIT_US

pytestmark = pytest.mark.gpu

from harness import NEAR_TIE, make_pair  # noqa: E402


def _c1(max_seq=64, seed=5, **kw):
    w = synth.WORKLOADS["C1"]
    sh = dataclasses.replace(w.shape, max_seq=max_seq)
    om, ctx, _ = make_pair(sh, seed, **kw)
    return w, sh, om, ctx


def test_expired_wait_returns_timeout_and_the_context_recovers():
    """The step kernel's first grid barrier waits for 149 arrivals of 148 CTAs and gives up after 3 ms: the launch ends by
    itself, the call reports CL_ETIMEOUT, nothing is committed, and after the setting is taken back the same context
    decodes correctly again."""
    w, sh, om, ctx = _c1()
    prompt = synth.make_prompt(2, 12, sh.vocab)
    first = ctx.cl_prefill(prompt)
    ctx.cl_set_skip_set([0, 3, 0, 0])
    good = ctx.cl_draft(3, want_logits=True)
    ctx.cl_rollback(len(prompt), first)
    ctx.cl_debug_set(CL_DEBUG_WAIT_LIMIT_US, 3000)
    ctx.cl_debug_set(CL_DEBUG_BARRIER_EXTRA, 1)
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_draft(3)
    assert e.value.code == 6 and "wait expired" in str(e.value)
    with pytest.raises(cl.ConfLayersError) as e:                       # vanilla steps run the same kernel
        ctx.cl_step_vanilla()
    assert e.value.code == 6
    ctx.cl_debug_set(CL_DEBUG_BARRIER_EXTRA, 0)
    ctx.cl_debug_set(CL_DEBUG_WAIT_LIMIT_US, 2_000_000)
    assert ctx.cl_prefill(prompt) == first
    again = ctx.cl_draft(3, want_logits=True)
    assert np.array_equal(again["tokens"], good["tokens"]) and np.array_equal(again["logits"], good["logits"])
    # and a fresh context is not affected by the old one's history
    _, _, _, ctx2 = _c1()
    assert ctx2.cl_prefill(prompt) == first


def test_expired_wait_in_the_row_pass_returns_timeout_and_the_context_recovers():
    """The same in the persistent T-row pass of a 16-bit model: its one grid barrier (in front of the LM-head merge) waits
    for one arrival too many and gives up after 3 ms; the launch winds down by itself (copies in flight awaited, tensor
    memory released), cl_verify reports CL_ETIMEOUT and commits nothing, and the next pass in the same context is correct."""
    w = synth.reduced(synth.WORKLOADS["C2"], n_layers=2, prompt_len=10, gen_len=4)
    sh = dataclasses.replace(w.shape, max_seq=64)
    om, ctx, _ = make_pair(sh, 8)
    prompt = synth.make_prompt(8, 10, sh.vocab)
    first = ctx.cl_prefill(prompt)
    ctx.cl_force_tokens([5, 6, 7])
    good = ctx.cl_verify(4, want_logits=True)
    ctx.cl_debug_set(CL_DEBUG_WAIT_LIMIT_US, 3000)
    ctx.cl_debug_set(CL_DEBUG_BARRIER_EXTRA, 1)
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_verify(4)
    assert e.value.code == 6
    assert ctx.cl_get_stats().ctx_len == len(prompt)
    ctx.cl_debug_set(CL_DEBUG_BARRIER_EXTRA, 0)
    ctx.cl_debug_set(CL_DEBUG_WAIT_LIMIT_US, 2_000_000)
    assert ctx.cl_prefill(prompt) == first
    ctx.cl_force_tokens([5, 6, 7])
    again = ctx.cl_verify(4, want_logits=True)
    assert np.array_equal(again["targets"], good["targets"]) and np.array_equal(again["logits"], good["logits"])


@pytest.mark.parametrize("name", ["C1", "C2"])
def test_error_flag_stops_verify_accept_and_prefill_from_committing(name):
    """A device-side error flag (what an expired wait leaves) found by cl_verify, cl_accept or cl_prefill makes the call
    return CL_ETIMEOUT; the cache length and the pending token stay as they were."""
    w0 = synth.WORKLOADS[name]
    w = synth.reduced(w0, n_layers=2, prompt_len=10, gen_len=4) if name != "C1" else w0
    sh = dataclasses.replace(w.shape, max_seq=64)
    om, ctx, _ = make_pair(sh, 6)
    prompt = synth.make_prompt(3, 10, sh.vocab)
    first = ctx.cl_prefill(prompt)
    ctx.cl_set_skip_set(np.zeros(sh.n_layers, np.uint8))
    d = ctx.cl_draft(2)
    ctx.cl_debug_set(CL_DEBUG_DEVICE_ERR, 4)
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_verify(3)
    assert e.value.code == 6
    assert ctx.cl_get_stats().ctx_len == len(prompt)
    v = ctx.cl_verify(3)                                               # the flag was cleared: the pass now goes through
    ctx.cl_debug_set(CL_DEBUG_DEVICE_ERR, 2)
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_accept()
    assert e.value.code == 6
    assert ctx.cl_get_stats().ctx_len == len(prompt)                   # nothing was committed
    n, em = ctx.cl_accept()
    assert 0 <= n <= 2 and list(em[:n]) == list(d["tokens"][:n]) and em[n] == v["targets"][n]
    ctx.cl_debug_set(CL_DEBUG_DEVICE_ERR, 1)
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_prefill(prompt)
    assert e.value.code == 6
    with pytest.raises(cl.ConfLayersError) as e:                       # the aborted prefill left no usable state
        ctx.cl_draft(2)
    assert e.value.code == 4
    assert ctx.cl_prefill(prompt) == first


def test_rollback_cannot_move_past_the_written_cache():
    w, sh, om, ctx = _c1()
    prompt = synth.make_prompt(4, 9, sh.vocab)
    first = ctx.cl_prefill(prompt)
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_rollback(10, first)
    assert e.value.code == 5 and "cache holds" in str(e.value)
    ctx.cl_rollback(9, first)
    ctx.cl_force_tokens([1, 2, 3])
    ctx.cl_verify(4)                                                   # writes positions 9..12 of every layer
    ctx.cl_rollback(13, first)
    with pytest.raises(cl.ConfLayersError):
        ctx.cl_rollback(14, first)
    ctx.cl_rollback(4, first)                                          # backwards is always allowed


def test_search_needs_a_tapped_prefill_and_a_full_window():
    w, sh, om, ctx = _c1(max_seq=128, tap_positions=32)
    prompt = synth.make_prompt(5, 8, sh.vocab)
    sel = cl.SelectCfg.make(w.lo, w.hi, n_skip=1)
    ctx.cl_prefill(prompt)                                             # no taps: the ring holds nothing of this input
    ctx.cl_set_skip_set([0, 3, 0, 0])
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_generate_search(3, 20, 2, 10.0, 2, sel)
    assert e.value.code == 4 and "tap_hidden" in str(e.value)
    ctx.cl_prefill(prompt, tap_hidden=True)                            # 8 prompt rows + 2 cycles < 32 positions
    with pytest.raises(cl.ConfLayersError) as e:
        ctx.cl_generate_search(3, 20, 2, 10.0, 2, sel)
    assert e.value.code == 4 and "of 32 positions" in str(e.value)


@pytest.mark.parametrize("name,L", [("C1", 4), ("C2", 3), ("C3", 2)])
def test_same_call_twice_gives_the_same_bits(name, L):
    """Every reduction runs in a fixed order, so repeating a call in one context repeats its bits: verify logits and
    targets, draft logits, generated tokens.  (Between two contexts the LM-head partial grouping of the step kernel can
    differ, because the row shares of its CTAs are measured at load.)"""
    w0 = synth.WORKLOADS[name]
    w = synth.reduced(w0, n_layers=L, prompt_len=33, gen_len=8)
    sh = dataclasses.replace(w.shape, max_seq=96)
    om, ctx, _ = make_pair(sh, w.seed + 1, gen_device="cuda" if name == "C3" else "cpu")
    prompt = synth.make_prompt(w.seed, 33, sh.vocab)
    mask = synth.layers_to_mask([1], L)
    runs = []
    for _ in range(2):
        first = ctx.cl_prefill(prompt)
        ctx.cl_set_skip_set(mask)
        d = ctx.cl_draft(4, want_logits=True)
        v = ctx.cl_verify(5, want_logits=True)
        n, em = ctx.cl_accept()
        toks, st = ctx.cl_generate(4, 24)
        runs.append((first, d["tokens"], d["logits"], d["conf"], d["p_max"], v["targets"], v["logits"], n, em, toks))
    for a, b in zip(*runs):
        assert np.array_equal(np.asarray(a), np.asarray(b))
