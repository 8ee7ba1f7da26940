"""Seeded synthetic inputs for the ConfLayers hot path.

This module only *makes inputs*: random-init Llama-style weights, random prompts,
random hidden states, synthetic round scores and the evenly spaced "fixed" skip
sets.  It holds none of the method's arithmetic (no transformer math, no
confidence, no selection) and is the one module that both the CPU oracle's
callers and the CUDA path's callers use, so that both sides see identical bits.

The five workload shapes mirror the paper's experimental set-up (Section 4.1:
Llama-family decoders, batch 1, greedy decoding, few-shot prompts of 10^2-10^3
tokens, at most 512 generated tokens).  Trained weights and the evaluation
datasets are not available, so weights are N(0, 0.02) and prompts are uniform
random token ids: only the shapes are taken from the paper.

Determinism: every tensor is drawn from its own ``torch.Generator`` seeded with
``seed * 1_000_003 + tensor_id``, in fp32, then rounded (RNE) to the storage
type.  The same call on the same device gives the same bits; the oracle and the
CUDA path are always handed the *same* tensors (host copies of them for the
oracle), so nothing depends on CPU and GPU generators agreeing.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    max_seq: int
    weight_dtype: str = "bf16"          # "bf16" | "fp16" | "fp32": storage type of weights, KV cache and taps
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    std: float = 0.02
    lm_head_scale: float = 1.0
    n_kv_heads: int = 0                 # key/value heads of grouped-query attention (0: same as n_heads)

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    @property
    def kv_heads(self) -> int:
        return self.n_kv_heads or self.n_heads


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    seed: int
    prompt_len: int
    gen_len: int
    K: tuple                 # draft lengths exercised
    lo: int                  # first eligible layer (inclusive)
    hi: int                  # last eligible layer (inclusive)
    n_skip_conf: int         # size of the confidence-selected skip set
    fixed_ratios: tuple = ()


def _shape(L, d, H, F, V, max_seq, wd="bf16", head_scale=1.0):
    return ModelShape(L, d, H, F, V, max_seq, wd, lm_head_scale=head_scale)


# The five workloads (tiny / 12-layer / 7B-shape / 13B-shape / all-layer scoring).
WORKLOADS: Dict[str, Workload] = {
    "C1": Workload("C1", _shape(4, 256, 4, 688, 1024, 128, "fp32"), 0, 16, 32, (4,), 1, 2, 1),
    "C2": Workload("C2", _shape(12, 768, 12, 2048, 32000, 320, "bf16", 4.0), 1, 128, 128, (4,), 1, 10, 3),
    "C3": Workload("C3", _shape(32, 4096, 32, 11008, 32000, 832, "bf16"), 2, 512, 256, (4, 8), 2, 29, 14,
                   (0.25, 0.5)),
    "C4": Workload("C4", _shape(40, 5120, 40, 13824, 32000, 1344, "bf16"), 3, 1024, 256, (6,), 1, 38, 15),
}

# All-layer confidence scoring workload: [layers, positions, d_model] hidden states
# through a shared [vocab, d_model] LM head, repeated for 8 search rounds.
C5 = dict(name="C5", n_layers=32, positions=64, d_model=4096, vocab=32000, seed=4, iters=8,
          rms_eps=1e-5, lo=2, hi=29, n_skip=14)


# tensor ids (per-tensor generator streams)
_T_EMBED, _T_HEAD, _T_LAYER0 = 1, 2, 16
_PER_LAYER = 8
_T_PROMPT, _T_HIDDEN0, _T_SCORES = 7, 4096, 9


def _gen(seed: int, tid: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + int(tid))
    return g


def _normal(shape, std, seed, tid, dtype, device) -> torch.Tensor:
    x = torch.randn(shape, generator=_gen(seed, tid, device), dtype=torch.float32, device=device)
    x.mul_(std)
    return x.to(dtype).contiguous()


def torch_dtype(weight_dtype: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}[weight_dtype]


def make_weights(shape: ModelShape, seed: int, device="cpu") -> Dict[str, object]:
    """Random-init Llama-style decoder weights, every matrix stored (out, in) row-major.

    Returns a dict: embed [V,d], lm_head [V,d], final_norm fp32[d], and per-layer lists
    wq, wo [d,d], wk, wv [kv_heads*head_dim, d], wg, wu [F,d], wd [d,F], norm1, norm2 fp32[d] (gains = 1).
    """
    dt = torch_dtype(shape.weight_dtype)
    L, d, F, V = shape.n_layers, shape.d_model, shape.d_ffn, shape.vocab
    w: Dict[str, object] = {
        "embed": _normal((V, d), shape.std, seed, _T_EMBED, dt, device),
        "lm_head": _normal((V, d), shape.std * shape.lm_head_scale, seed, _T_HEAD, dt, device),
        "final_norm": torch.ones(d, dtype=torch.float32, device=device),
    }
    kvd = shape.kv_heads * shape.head_dim
    names = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")
    dims = ((d, d), (kvd, d), (kvd, d), (d, d), (F, d), (F, d), (d, F))
    for n in names + ("norm1", "norm2"):
        w[n] = []
    for l in range(L):
        for j, (n, sh) in enumerate(zip(names, dims)):
            w[n].append(_normal(sh, shape.std, seed, _T_LAYER0 + l * _PER_LAYER + j, dt, device))
        w["norm1"].append(torch.ones(d, dtype=torch.float32, device=device))
        w["norm2"].append(torch.ones(d, dtype=torch.float32, device=device))
    return w


def damp_output_projections(w: Dict[str, object], layers, factor: float) -> Dict[str, object]:
    """Scales, in place, the attention output projection and the FFN down projection of the given layers by `factor`
    (and rounds back to the storage type): those layers then add little to the residual stream, which is what a
    trained model's skippable layers look like to the draft model.  Random-init layers all matter equally, so a model
    made by ``make_weights`` alone accepts almost no draft once layers are skipped."""
    for l in layers:
        for n in ("wo", "wd"):
            t = w[n][int(l)]
            w[n][int(l)] = (t.float() * factor).to(t.dtype).contiguous()
    return w


def weights_to(w: Dict[str, object], device) -> Dict[str, object]:
    """Copy a weight dict to another device (bit-identical values)."""
    out: Dict[str, object] = {}
    for k, v in w.items():
        out[k] = [t.to(device) for t in v] if isinstance(v, list) else v.to(device)
    return out


def make_prompt(seed: int, n: int, vocab: int) -> np.ndarray:
    """Uniform random token ids, int32[n]."""
    g = _gen(seed, _T_PROMPT, "cpu")
    return torch.randint(0, vocab, (n,), generator=g, dtype=torch.int64).to(torch.int32).numpy()


def make_hidden(seed: int, stream: int, n_layers: int, positions: int, d_model: int, device="cpu") -> torch.Tensor:
    """Hidden states ~N(0,1), bf16 [n_layers, positions, d_model]; one tensor per search round."""
    return _normal((n_layers, positions, d_model), 1.0, seed, _T_HIDDEN0 + stream, torch.bfloat16, device)


def make_lm_head(seed: int, vocab: int, d_model: int, std: float = 0.02, device="cpu") -> torch.Tensor:
    return _normal((vocab, d_model), std, seed, _T_HEAD, torch.bfloat16, device)


def make_round_scores(seed: int, iters: int) -> np.ndarray:
    """Synthetic per-round scores (stand-in for the mean accepted tokens of a search round), fp32[iters]."""
    g = _gen(seed, _T_SCORES, "cpu")
    return (1.0 + 8.0 * torch.rand((iters,), generator=g, dtype=torch.float32)).numpy()


def uniform_skip_layers(lo: int, hi: int, n_skip: int) -> List[int]:
    """Evenly spaced whole-layer skip set inside the eligible range [lo, hi] (the uniformly
    skipped initial draft model of Section 3, and the workloads' fixed 25 % / 50 % sets)."""
    n_e = hi - lo + 1
    if n_skip <= 0:
        return []
    if n_skip > n_e:
        raise ValueError("n_skip exceeds the eligible range")
    return sorted({lo + ((j + 1) * n_e) // n_skip - 1 for j in range(n_skip)})


def layers_to_mask(layers, n_layers: int) -> np.ndarray:
    """uint8[L] mask: 3 = whole layer skipped (bit0 attention, bit1 FFN), 0 = kept."""
    m = np.zeros(n_layers, dtype=np.uint8)
    for l in layers:
        m[int(l)] = 3
    return m


def n_skip_for_ratio(lo: int, hi: int, ratio: float) -> int:
    return int(np.floor(ratio * (hi - lo + 1) + 0.5))


def reduced(w: Workload, n_layers: Optional[int] = None, prompt_len: Optional[int] = None,
            gen_len: Optional[int] = None, max_seq: Optional[int] = None) -> Workload:
    """A smaller case of the same shape family (fewer layers / shorter run) for oracle-speed parity tests."""
    sh = w.shape
    L = n_layers or sh.n_layers
    p = prompt_len or w.prompt_len
    g = gen_len or w.gen_len
    ms = max_seq or (p + g + 16 + max(w.K))
    sh2 = dataclasses.replace(sh, n_layers=L, max_seq=ms)
    hi = min(w.hi, L - 2) if L >= 3 else 0
    lo = min(w.lo, hi)
    n_e = hi - lo + 1
    return dataclasses.replace(w, name=f"{w.name}-L{L}-p{p}-g{g}", shape=sh2, prompt_len=p, gen_len=g,
                               lo=lo, hi=hi, n_skip_conf=max(1, min(w.n_skip_conf, n_e // 2)))
