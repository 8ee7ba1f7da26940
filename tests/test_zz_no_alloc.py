"""The allocation-free scoring call against the context's own scoring call (run on a B200).

cl_layer_confidences_static() is for processes in which this library must not allocate device
memory (the GPU is already fully reserved by the host framework's allocator, or a cudaMalloc's
device-wide synchronisation is not acceptable inside the serving loop).  It keeps all of its working
memory in one fixed array inside the library, so the thing to check is that a call gives the same
confidences as cl_layer_confidences() and that a second call, which finds the first call's leftovers
in that array, still does.  This file sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_14612_b200 as cl
import synth

pytestmark = pytest.mark.gpu

TOL = 1e-2          # max-abs tolerance on confidences and probabilities, as in the other parity tests
NEAR_TIE = 1e-2     # a differing greedy token is tolerated only below this top-2 logit margin


def _check(got, want, hidden, head, gain, eps):
    assert np.abs(got["conf"] - want["conf"]).max() <= TOL
    assert np.abs(got["p_max"] - want["p_max"]).max() <= TOL
    diff = np.argwhere(got["argmax"] != want["argmax"])
    for r, p in diff:                                   # only a near tie may decide the token differently
        h = hidden[r, p].double().cpu()
        x = h * torch.rsqrt((h * h).mean() + eps) * gain.double().cpu()
        top = torch.topk(head.double().cpu() @ x, 2).values
        assert float(top[0] - top[1]) < NEAR_TIE, (r, p)


@pytest.mark.parametrize("dtype,V,d", [("bf16", 5003, 1024), ("fp32", 1024, 256)])
def test_static_scoring_matches_context_scoring_twice(dtype, V, d):
    dt = synth.torch_dtype(dtype)
    rows, P = 3, 7                                      # 21 rows: two full passes of 8 and a ragged one of 5
    g = torch.Generator(device="cuda").manual_seed(11)
    head = (0.05 * torch.randn((V, d), generator=g, device="cuda")).to(dt).contiguous()
    gain = (1.0 + 0.1 * torch.randn((d,), generator=g, device="cuda")).float().contiguous()
    ctx = cl.Context(rows, d, d // 64, 64, V, 8, dtype)
    ctx.cl_load(dict(lm_head=head, final_norm=gain), head_only=True)
    for call in range(2):                               # the second call meets the first one's scratch contents
        hidden = (1.0 + call) * torch.randn((rows, P, d), generator=g, device="cuda")
        hidden = hidden.to(dt).contiguous()
        want = ctx.cl_layer_confidences(hidden)
        got = cl.cl_layer_confidences_static(head, gain, hidden, rms_eps=1e-5)
        _check(got, want, hidden, head, gain, 1e-5)
        assert (got["conf"] > -1e-6).all() and (got["conf"] < 1 + 1e-6).all()
        # and against the CPU oracle's Eq. 1-4 on the same rows (the context's call runs different kernels for a
        # 16-bit head, so the comparison above is a real one, but this one does not lean on the library at all)
        o = oracle.layer_confidences(hidden.cpu(), head.cpu(), gain.cpu(), 1e-5)
        assert np.abs(got["conf"] - o["conf"]).max() <= TOL
        assert np.abs(got["p_max"] - o["p_max"]).max() <= TOL
        assert not ((got["argmax"] != o["argmax"]) & (o["margin"] >= NEAR_TIE)).any()


def test_static_scoring_rejects_sizes_beyond_its_fixed_scratch():
    head = torch.zeros((16, 64), device="cuda")
    gain = torch.ones(64, device="cuda")
    too_many = torch.zeros((4097, 64), device="cuda")
    with pytest.raises(cl.ConfLayersError) as e:
        cl.cl_layer_confidences_static(head, gain, too_many)
    assert e.value.code == 5 and "4096" in str(e.value)
    wide = torch.zeros((2, 8200), device="cuda")
    with pytest.raises(cl.ConfLayersError) as e:
        cl.cl_layer_confidences_static(torch.zeros((16, 8200), device="cuda"), torch.ones(8200, device="cuda"), wide)
    assert e.value.code == 5


def test_static_scoring_rejects_unsupported_dtype_shape_and_alignment():
    """These fail on the host and launch nothing: an fp16 head (the call knows fp32 and bf16 only), a hidden tensor or a
    gain whose width is not d_model, and -- through the raw C call -- a pointer that is not 16-byte aligned."""
    head16 = torch.zeros((16, 64), device="cuda", dtype=torch.float16)
    gain = torch.ones(64, device="cuda")
    with pytest.raises(ValueError):
        cl.cl_layer_confidences_static(head16, gain, torch.zeros((2, 64), device="cuda", dtype=torch.float16))
    head = torch.zeros((16, 64), device="cuda")
    with pytest.raises(ValueError):
        cl.cl_layer_confidences_static(head, gain, torch.zeros((2, 32), device="cuda"))
    with pytest.raises(ValueError):
        cl.cl_layer_confidences_static(head, torch.ones(32, device="cuda"), torch.zeros((2, 64), device="cuda"))
    lib = cl.load_library()
    hidden = torch.zeros((3, 64), device="cuda")
    out = np.zeros(2, np.float32)
    rc = lib.cl_layer_confidences_static(head.data_ptr(), gain.data_ptr(), 16, 64, 2, 1e-5, hidden.data_ptr(), 2, None,
                                         out.ctypes.data, None, None)
    assert rc == 1 and b"weight_dtype" in lib.cl_last_error(None)
    rc = lib.cl_layer_confidences_static(head.data_ptr(), gain.data_ptr(), 16, 64, 0, 1e-5, hidden.data_ptr() + 4, 2, None,
                                         out.ctypes.data, None, None)
    assert rc == 1 and b"16-byte aligned" in lib.cl_last_error(None)
