"""How far the CUDA path may sit from the oracle at full depth, and why (run on a B200).

The KV cache and the hidden-state taps are stored in bf16.  A key or value whose fp32 value lies within rounding noise
of a bf16 boundary is rounded to different neighbours by two correct implementations; that element then differs by
2^-9 relative, and the difference travels through the remaining layers.  So the distance between two correct
implementations grows with depth and cannot be held to the 1e-2 that is kept wherever the depth is at most 12 layers.
This file measures the floor with a reference that shares nothing with either side -- the same Llama forward pass
written with library tensor operations in fp64, without any rounding of the cache -- and holds the CUDA path to bounds
that are 1.5 x the distances measured when the test was written, depth by depth, instead of one blanket tolerance."""
import dataclasses
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2604_14612_b200 as cl
import synth

pytestmark = pytest.mark.gpu

from harness import make_pair  # noqa: E402


def fp64_logits(shape, W, tokens, kv_round=None):
    """Llama forward over `tokens` from an empty cache with library tensor ops in fp64 on the GPU; logits [n, V].
    kv_round (a torch dtype) rounds keys (after the rotary embedding) and values to that type, as a cache would."""
    dev = "cuda"
    d, H, hd = shape.d_model, shape.n_heads, shape.d_model // shape.n_heads
    n = len(tokens)
    f = lambda t: t.to(dev).double()
    x = f(W["embed"])[torch.as_tensor(np.asarray(tokens, np.int64), device=dev)]
    pos = torch.arange(n, device=dev, dtype=torch.float64)
    inv = shape.rope_theta ** (-torch.arange(0, hd, 2, device=dev, dtype=torch.float64) / hd)
    ang = pos[:, None] * inv[None, :]
    cos, sin = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]

    def norm(v, g):
        return v * torch.rsqrt((v * v).mean(-1, keepdim=True) + shape.rms_eps) * f(g)

    def rope(v):   # [n, H, hd], pairs (i, i + hd / 2)
        a, b = v[..., :hd // 2], v[..., hd // 2:]
        return torch.cat([a * cos - b * sin, b * cos + a * sin], -1)

    causal = torch.tril(torch.ones(n, n, device=dev, dtype=torch.bool))
    for l in range(shape.n_layers):
        r = norm(x, W["norm1"][l])
        q = rope((r @ f(W["wq"][l]).T).view(n, H, hd))
        k = rope((r @ f(W["wk"][l]).T).view(n, H, hd))
        v = (r @ f(W["wv"][l]).T).view(n, H, hd)
        if kv_round is not None:
            k, v = k.to(kv_round).double(), v.to(kv_round).double()
        s = torch.einsum("ihd,jhd->hij", q, k) / hd ** 0.5
        s = s.masked_fill(~causal[None], float("-inf"))
        att = torch.einsum("hij,jhd->ihd", torch.softmax(s, -1), v).reshape(n, d)
        x = x + att @ f(W["wo"][l]).T
        r = norm(x, W["norm2"][l])
        g_ = r @ f(W["wg"][l]).T
        x = x + (torch.nn.functional.silu(g_) * (r @ f(W["wu"][l]).T)) @ f(W["wd"][l]).T
    return (norm(x, W["final_norm"]) @ f(W["lm_head"]).T).cpu().numpy()


# (shape, depth) -> (bound on |oracle - fp64|, bound on |CUDA pass - oracle|): 1.5 x the largest distances measured when
# this test was written.  7B layer shape at 8 / 16 / 32 layers: oracle 4.7e-2 / 7.3e-2 / 9.5e-2 from the exact result, which
# is also where rounding the cache alone puts an exact computation (4.7e-2 / 7.6e-2 / 9.3e-2); CUDA pass 5.3e-3 / 9.3e-3 /
# 1.4e-2 from the oracle here and 1.6e-2 in the full-depth lock-step test.  13B shape at its 40 layers: 1.35e-1 (floor
# 1.38e-1) and 2.4e-2 / 2.6e-2.  With one tensor-core accumulation chain over all of K instead of a drain into fp32
# registers every four ring slots the CUDA pass sat twice as far from the oracle (1.1e-2 / 1.5e-2 / 2.7e-2).
BOUNDS = {("C3", 8): (7.0e-2, 8.0e-3), ("C3", 16): (1.1e-1, 1.4e-2), ("C3", 32): (1.45e-1, 2.4e-2), ("C4", 40): (2.0e-1, 3.9e-2)}


@pytest.mark.parametrize("name,L", [("C3", 8), ("C3", 16), ("C3", 32), ("C4", 40)])
def test_distance_to_the_oracle_grows_with_depth_as_the_storage_format_dictates(name, L):
    w = synth.reduced(synth.WORKLOADS[name], n_layers=L, prompt_len=12, gen_len=4)
    om, ctx, Wh = make_pair(w.shape, w.seed, gen_device="cuda")
    prompt = synth.make_prompt(w.seed, w.prompt_len, w.shape.vocab)
    rows = [int(t) for t in prompt[8:]]                               # verify rows: the last four prompt tokens
    # CUDA: eight prompt tokens through the prompt pass, then one 4-row verify pass
    first = ctx.cl_prefill(prompt[:8])
    ctx.cl_rollback(8, rows[0])
    ctx.cl_force_tokens(rows[1:])
    got = ctx.cl_verify(4, want_logits=True)["logits"]
    # oracle: the same rows on its own cache
    om.forward(prompt[:8], 0, want_logits=False)
    want = om.forward(rows, 8)["logits"]
    W = synth.make_weights(w.shape, w.seed, device="cuda")
    exact = fp64_logits(w.shape, W, prompt)[8:]
    rounded = fp64_logits(w.shape, W, prompt, kv_round=torch.bfloat16)[8:]
    d_oracle = float(np.abs(want - exact).max())
    d_round = float(np.abs(rounded - exact).max())                    # what rounding the cache alone does to an exact computation
    d_cuda = float(np.abs(got - want).max())
    d_cuda_exact = float(np.abs(got - exact).max())
    part = np.partition(want.astype(np.float64), -2, axis=1)
    near = int(((part[:, -1] - part[:, -2]) < d_cuda).sum())
    print(f"{name} depth {L}: |oracle - fp64| {d_oracle:.2e}  |fp64 with bf16 cache - fp64| {d_round:.2e}  |CUDA - oracle| {d_cuda:.2e}  "
          f"|CUDA - fp64| {d_cuda_exact:.2e}  rows whose top-2 margin is below that distance: {near} of {len(rows)}  "
          f"(chain {os.environ.get('CL_ROWS_CHAIN', 'default')})")
    b_oracle, b_cuda = BOUNDS[(name, L)]
    assert d_oracle <= b_oracle, "the oracle moved away from the fp64 reference"
    assert d_cuda <= b_cuda, "the CUDA pass moved away from the oracle"
    # both sit as far from the exact result as rounding the cache alone puts an exact computation (measured ratios 0.97 to
    # 1.04), and from each other a small fraction of that (0.11 to 0.15)
    assert d_oracle <= 1.5 * d_round and d_cuda_exact <= 1.5 * d_round
    assert d_cuda <= 0.3 * d_round
