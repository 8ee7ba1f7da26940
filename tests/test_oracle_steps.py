"""Pins for the CPU oracle's elementary steps and its transformer forward.

Each check compares the oracle with something other than itself: a closed form, an identity the
operation must satisfy, a brute-force evaluation, or an independent library implementation of the
same architecture (Hugging Face's LlamaForCausalLM in fp64).
"""
import ctypes as C
import math

import numpy as np
import pytest
import torch

import oracle
import synth
from oracle.model import _ptr, lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def test_round_bf16_matches_torch():
    g = torch.Generator().manual_seed(5)
    x = torch.randn(4096, generator=g) * torch.logspace(-6, 6, 4096)
    want = x.to(torch.bfloat16).float().numpy()
    got = np.array([lib().orc_round_bf16(float(v)) for v in x.numpy()], np.float32)
    assert np.array_equal(want, got)
    # ties go to even: 1 + 2^-8 is halfway between bf16(1.0) and bf16(1.0078125)
    assert lib().orc_round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert lib().orc_round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6


def test_rmsnorm_closed_form():
    x, g, out = _f32([3, 4]), _f32([1, 2]), np.empty(2, np.float32)
    lib().orc_rmsnorm(_ptr(x), _ptr(g), 2, 0.0, _ptr(out))
    rms = math.sqrt(12.5)
    assert np.allclose(out, [3 / rms, 8 / rms], rtol=1e-7)
    # eps enters under the root: x = 0 gives 0, and a huge eps scales down
    x = _f32([2, 2, 2, 2]); g = _f32([1, 1, 1, 1]); out = np.empty(4, np.float32)
    lib().orc_rmsnorm(_ptr(x), _ptr(g), 4, 5.0, _ptr(out))
    assert np.allclose(out, 2 / 3.0, rtol=1e-7)


def test_silu_values():
    assert lib().orc_silu(0.0) == 0.0
    assert abs(lib().orc_silu(1.0) - 0.7310585786300049) < 1e-15
    assert abs(lib().orc_silu(-1.0) + 0.2689414213699951) < 1e-15
    assert abs(lib().orc_silu(30.0) - 30.0) < 1e-11


def test_rope_identities():
    hd = 64
    rng = np.random.default_rng(0)
    v = _f32(rng.standard_normal(hd))
    a = v.copy()
    lib().orc_rope(_ptr(a), hd, 0, 10000.0)
    assert np.array_equal(a, v)                                   # position 0 is the identity
    a = v.copy()
    lib().orc_rope(_ptr(a), hd, 37, 10000.0)
    assert abs(np.linalg.norm(a) - np.linalg.norm(v)) < 1e-5      # rotations keep the norm
    # pair (0, hd/2) rotates by exactly `pos` radians (frequency of index 0 is 1)
    e = np.zeros(hd, np.float32); e[0] = 1.0
    lib().orc_rope(_ptr(e), hd, 3, 10000.0)
    assert abs(e[0] - math.cos(3.0)) < 1e-7 and abs(e[hd // 2] - math.sin(3.0)) < 1e-7
    # the last pair turns by pos * theta^(-(hd-2)/hd)
    e = np.zeros(hd, np.float32); e[hd // 2 - 1] = 1.0
    lib().orc_rope(_ptr(e), hd, 1000, 10000.0)
    ang = 1000 * 10000.0 ** (-(hd - 2) / hd)
    assert abs(e[hd // 2 - 1] - math.cos(ang)) < 1e-7 and abs(e[hd - 1] - math.sin(ang)) < 1e-7
    # relative-position property: <rope(q,m), rope(k,n)> depends on m - n only
    q, k = _f32(rng.standard_normal(hd)), _f32(rng.standard_normal(hd))
    def dot_at(m, n):
        qq, kk = q.copy(), k.copy()
        lib().orc_rope(_ptr(qq), hd, m, 10000.0); lib().orc_rope(_ptr(kk), hd, n, 10000.0)
        return float(np.dot(qq.astype(np.float64), kk.astype(np.float64)))
    assert abs(dot_at(9, 4) - dot_at(105, 100)) < 1e-4
    assert abs(dot_at(9, 4) - dot_at(4, 9)) > 1e-3               # and it is not symmetric


def test_attention_special_cases():
    hd, stride = 8, 16
    rng = np.random.default_rng(1)
    q = _f32(rng.standard_normal(hd))
    k = _f32(rng.standard_normal((5, stride)))
    v = _f32(rng.standard_normal((5, stride)))
    out = np.empty(hd, np.float32)
    lib().orc_attention_head(_ptr(q), _ptr(k), _ptr(v), 1, hd, stride, _ptr(out))
    assert np.array_equal(out, v[0, :hd])                         # one key: returns its value
    k2 = np.repeat(k[:1], 5, axis=0).copy()
    lib().orc_attention_head(_ptr(q), _ptr(k2), _ptr(v), 5, hd, stride, _ptr(out))
    assert np.allclose(out, v[:, :hd].mean(axis=0), atol=1e-6)    # equal keys: plain mean of values
    # general case against a float64 numpy softmax
    lib().orc_attention_head(_ptr(q), _ptr(k), _ptr(v), 5, hd, stride, _ptr(out))
    s = (k[:, :hd].astype(np.float64) @ q.astype(np.float64)) / math.sqrt(hd)
    p = np.exp(s - s.max()); p /= p.sum()
    assert np.allclose(out, p @ v[:, :hd].astype(np.float64), atol=1e-6)


def test_dot_row_exact_small_integers_and_bf16():
    W = _f32(np.arange(12).reshape(3, 4))
    x = _f32([1, -2, 3, -4])
    assert lib().orc_dot_row(_ptr(W), 0, 2, 4, _ptr(x)) == float(8 - 18 + 30 - 44)
    Wb = torch.tensor(W).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert lib().orc_dot_row(_ptr(Wb), 1, 1, 4, _ptr(x)) == float(4 - 10 + 18 - 28)
    out = np.empty((2, 3), np.float32)
    xs = _f32([[1, 0, 0, 0], [0, 0, 0, 1]])
    lib().orc_matmul_rows(_ptr(W), 0, 3, 4, _ptr(xs), 2, _ptr(out))
    assert np.array_equal(out, [[0, 4, 8], [3, 7, 11]])           # picks columns 0 and 3, not transposed


def _hf_model(shape, W):
    tr = pytest.importorskip("transformers")
    cfg = tr.LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
                         num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
                         num_key_value_heads=shape.n_heads, rms_norm_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                         max_position_embeddings=shape.max_seq, tie_word_embeddings=False, attention_bias=False,
                         mlp_bias=False, hidden_act="silu")
    hf = tr.LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": W["embed"], "lm_head.weight": W["lm_head"], "model.norm.weight": W["final_norm"]}
    names = dict(wq="self_attn.q_proj", wk="self_attn.k_proj", wv="self_attn.v_proj", wo="self_attn.o_proj",
                 wg="mlp.gate_proj", wu="mlp.up_proj", wd="mlp.down_proj", norm1="input_layernorm",
                 norm2="post_attention_layernorm")
    for l in range(shape.n_layers):
        for k, n in names.items():
            sd[f"model.layers.{l}.{n}.weight"] = W[k][l]
    res = hf.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not res.unexpected_keys and all("rotary" in k for k in res.missing_keys)
    return hf


def test_forward_matches_library_llama_fp64():
    """The whole transformer step against an independent library implementation of the same
    architecture, with non-trivial norm gains so a dropped gain would show."""
    w = synth.WORKLOADS["C1"]
    sh = w.shape
    W = synth.make_weights(sh, w.seed)
    g = torch.Generator().manual_seed(11)
    W["final_norm"] = 1.0 + 0.3 * torch.randn(sh.d_model, generator=g)
    for l in range(sh.n_layers):
        W["norm1"][l] = 1.0 + 0.3 * torch.randn(sh.d_model, generator=g)
        W["norm2"][l] = 1.0 + 0.3 * torch.randn(sh.d_model, generator=g)
    hf = _hf_model(sh, W)
    prompt = synth.make_prompt(3, 24, sh.vocab)
    with torch.no_grad():
        ref = hf(torch.tensor(prompt[None].astype(np.int64)), output_hidden_states=True)
    m = oracle.OracleModel(sh, W)
    out = m.forward(prompt, 0, want_hidden=True)
    assert np.abs(out["logits"] - ref.logits[0].numpy()).max() < 2e-6
    # layer outputs (residual stream after the FFN add) = the library's hidden_states[l+1]
    # (its last entry has the final norm applied, so stop one short)
    for l in range(sh.n_layers - 1):
        assert np.abs(out["hid_ffn"][l] - ref.hidden_states[l + 1][0].numpy()).max() < 2e-6
    # cached decoding: prefix then one token at a time reproduces the same logits
    m2 = oracle.OracleModel(sh, W)
    m2.forward(prompt[:20], 0, want_logits=False)
    for t in range(20, 24):
        lg = m2.forward(prompt[t:t + 1], t)["logits"][0]
        assert np.abs(lg - ref.logits[0, t].numpy()).max() < 2e-6


def test_forward_rows_bitwise_independent_of_batching():
    """Row t of an n-row pass has the same bits as a one-row pass (what makes verify == vanilla exact)."""
    w = synth.WORKLOADS["C1"]
    W = synth.make_weights(w.shape, w.seed)
    p = synth.make_prompt(1, 12, w.shape.vocab)
    a = oracle.OracleModel(w.shape, W).forward(p, 0, want_hidden=True)
    m = oracle.OracleModel(w.shape, W)
    for t in range(12):
        b = m.forward(p[t:t + 1], t, want_hidden=True)
        assert np.array_equal(a["logits"][t], b["logits"][0])
        assert np.array_equal(a["hid_ffn"][:, t], b["hid_ffn"][:, 0])
        assert np.array_equal(a["hid_attn"][:, t], b["hid_attn"][:, 0])


def test_zero_output_projections_reduce_to_embedding_head():
    w = synth.WORKLOADS["C1"]
    sh = w.shape
    W = synth.make_weights(sh, w.seed)
    for l in range(sh.n_layers):
        W["wo"][l] = torch.zeros_like(W["wo"][l])
        W["wd"][l] = torch.zeros_like(W["wd"][l])
    m = oracle.OracleModel(sh, W)
    tok = np.array([5, 900], np.int32)
    lg = m.forward(tok, 0)["logits"]
    e = W["embed"][tok.astype(np.int64)].double()
    r = e / torch.sqrt((e * e).mean(dim=1, keepdim=True) + sh.rms_eps)
    want = (r @ W["lm_head"].double().T).numpy()
    assert np.abs(lg - want).max() < 1e-6


def test_skipped_layer_leaves_stream_and_cache_untouched():
    w = synth.WORKLOADS["C1"]
    sh = w.shape
    W = synth.make_weights(sh, w.seed)
    p = synth.make_prompt(2, 6, sh.vocab)
    mask = synth.layers_to_mask([2], sh.n_layers)
    m = oracle.OracleModel(sh, W)
    out = m.forward(p, 0, mask, want_hidden=True)
    assert np.all(m.read_kv(2, 0, 3) == 0) and np.all(m.read_kv(2, 1, 3) == 0)
    assert np.any(m.read_kv(1, 0, 3) != 0)
    # layer 3's input is layer 1's output: compare with a 3-layer model made of layers 0, 1, 3
    import dataclasses
    sh3 = dataclasses.replace(sh, n_layers=3)
    W3 = dict(W)
    for k in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2"):
        W3[k] = [W[k][0], W[k][1], W[k][3]]
    lg3 = oracle.OracleModel(sh3, W3).forward(p, 0)["logits"]
    assert np.array_equal(out["logits"], lg3)


def test_half_layer_skips_equal_zeroed_output_projections():
    """Skipping only the attention (FFN) half of a layer gives the logits of the model whose attention output
    (FFN down) projection in that layer is zero; the skipped attention half leaves its KV entries untouched."""
    w = synth.WORKLOADS["C1"]
    sh = w.shape
    W = synth.make_weights(sh, w.seed)
    p = synth.make_prompt(3, 7, sh.vocab)
    for bits, key in ((1, "wo"), (2, "wd")):
        mask = np.zeros(sh.n_layers, np.uint8)
        mask[1] = bits
        m = oracle.OracleModel(sh, W)
        got = m.forward(p, 0, mask)["logits"]
        kv_touched = bool(np.any(m.read_kv(1, 0, 2) != 0))
        assert kv_touched == (bits == 2)
        Wz = dict(W)
        Wz[key] = [t if l != 1 else torch.zeros_like(t) for l, t in enumerate(W[key])]
        want = oracle.OracleModel(sh, Wz).forward(p, 0)["logits"]
        assert np.array_equal(got, want)
    both = np.zeros(sh.n_layers, np.uint8)
    both[1] = 3
    m1 = oracle.OracleModel(sh, W).forward(p, 0, both)["logits"]
    Wz = dict(W)
    for key in ("wo", "wd"):
        Wz[key] = [t if l != 1 else torch.zeros_like(t) for l, t in enumerate(W[key])]
    assert np.array_equal(m1, oracle.OracleModel(sh, Wz).forward(p, 0)["logits"])


def test_bf16_storage_rounds_cache_and_taps():
    import dataclasses
    sh = dataclasses.replace(synth.WORKLOADS["C1"].shape, weight_dtype="bf16")
    W = synth.make_weights(sh, 7)
    m = oracle.OracleModel(sh, W)
    out = m.forward(synth.make_prompt(7, 5, sh.vocab), 0, want_hidden=True)
    k = m.read_kv(1, 0, 2)
    assert np.array_equal(k, torch.tensor(k).to(torch.bfloat16).float().numpy()) and np.any(k != 0)
    h = out["hid_ffn"]
    assert np.array_equal(h, torch.tensor(h).to(torch.bfloat16).float().numpy())


def test_round_fp16_and_widening_match_numpy_float16():
    """The oracle's binary16 rounding and widening are written from the format's definition; numpy's float16 is an
    independent implementation of the same format: random values over the whole range (subnormals, overflow), every
    one of the 65536 bit patterns, and the tie cases."""
    g = torch.Generator().manual_seed(6)
    x = (torch.randn(8192, generator=g) * torch.logspace(-9, 6, 8192)).numpy().astype(np.float32)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).astype(np.float32)
    got = np.array([lib().orc_round_fp16(float(v)) for v in x], np.float32)
    assert np.array_equal(want, got)
    bits = np.arange(65536, dtype=np.uint16)
    wide = bits.view(np.float16).astype(np.float32)
    mine = np.array([lib().orc_fp16_bits_to_f32(int(b)) for b in bits], np.float32)
    ok = np.isfinite(wide)
    assert np.array_equal(wide[ok], mine[ok]) and np.array_equal(np.isnan(wide), np.isnan(mine))
    assert np.array_equal(np.isinf(wide), np.isinf(mine))
    # ties to even: 1 + 2^-11 is halfway between 1 and 1 + 2^-10; 2^-25 is halfway between 0 and the smallest subnormal
    assert lib().orc_round_fp16(1.0 + 2.0 ** -11) == 1.0
    assert lib().orc_round_fp16(1.0 + 3 * 2.0 ** -11) == 1.0 + 2.0 ** -9
    assert lib().orc_round_fp16(2.0 ** -25) == 0.0 and lib().orc_round_fp16(3 * 2.0 ** -25) == 2.0 ** -23
    assert lib().orc_round_fp16(65519.0) == 65504.0 and np.isinf(lib().orc_round_fp16(65520.0))


def test_fp16_storage_rounds_cache_and_taps_and_reads_weights_exactly():
    import dataclasses
    sh = dataclasses.replace(synth.WORKLOADS["C1"].shape, weight_dtype="fp16")
    W = synth.make_weights(sh, 7)
    m = oracle.OracleModel(sh, W)
    out = m.forward(synth.make_prompt(7, 5, sh.vocab), 0, want_hidden=True)
    k = m.read_kv(1, 0, 2)
    assert np.array_equal(k, torch.tensor(k).to(torch.float16).float().numpy()) and np.any(k != 0)
    h = out["hid_ffn"]
    assert np.array_equal(h, torch.tensor(h).to(torch.float16).float().numpy())
    # the same model with its fp16 weights widened to fp32 differs only by the storage rounding of the cache
    # (relative 2^-11 per cached value): the weights are read exactly
    sh32 = dataclasses.replace(sh, weight_dtype="fp32")
    W32 = {n: ([t.float() for t in v] if isinstance(v, list) else v.float()) for n, v in W.items()}
    one = synth.make_prompt(7, 1, sh.vocab)
    a = oracle.OracleModel(sh, W).forward(one, 0)["logits"]
    b = oracle.OracleModel(sh32, W32).forward(one, 0)["logits"]
    assert np.abs(a - b).max() < 1e-3 and not np.array_equal(a, b)


def test_bad_arguments_are_rejected():
    w = synth.WORKLOADS["C1"]
    m = oracle.OracleModel(w.shape, synth.make_weights(w.shape, w.seed))
    with pytest.raises(ValueError):
        m.forward([w.shape.vocab], 0)
    with pytest.raises(ValueError):
        m.forward([1, 2], w.shape.max_seq - 1)


def test_grouped_query_attention_equals_replicated_kv_heads():
    """A model with n_kv_heads < n_heads gives the logits of the multi-head model whose K and V projections repeat
    every key/value head for its group of query heads; n_kv_heads = n_heads is the multi-head model itself."""
    import dataclasses
    w = synth.WORKLOADS["C1"]
    sh_g = dataclasses.replace(w.shape, n_kv_heads=2)          # 4 query heads, 2 key/value heads
    Wg = synth.make_weights(sh_g, 7)
    hd, group = sh_g.head_dim, sh_g.n_heads // 2
    Wm = dict(Wg)
    for key in ("wk", "wv"):
        Wm[key] = [t.view(2, hd, -1).repeat_interleave(group, dim=0).reshape(sh_g.d_model, -1).contiguous() for t in Wg[key]]
    p = synth.make_prompt(4, 9, sh_g.vocab)
    mask = synth.layers_to_mask([2], sh_g.n_layers)
    got = oracle.OracleModel(sh_g, Wg).forward(p, 0, mask)["logits"]
    want = oracle.OracleModel(w.shape, Wm).forward(p, 0, mask)["logits"]
    assert np.array_equal(got, want)
    same = oracle.OracleModel(dataclasses.replace(w.shape, n_kv_heads=w.shape.n_heads), Wm).forward(p, 0, mask)["logits"]
    assert np.array_equal(same, want)
    assert oracle.OracleModel(sh_g, Wg).read_kv(0, 0, 0).shape[0] == 2 * hd
