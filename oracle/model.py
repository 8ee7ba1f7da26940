"""ctypes loader and thin wrapper for the C oracle (test infrastructure only)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conflayers_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_LOCK = threading.Lock()
_LIB = None

CLAMP = 1.0e4      # logit clamp bound applied after the FP32 cast (Section 3.1; the paper gives no bound)
EPS_H = 1.0e-10    # epsilon inside the log of Eq. 2 (the paper gives no value)


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab", "max_seq")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("weight_dtype", C.c_int), ("n_kv_heads", C.c_int)]


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction) if missing or stale."""
    with _LOCK:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


def lib():
    global _LIB
    if _LIB is None:
        L = C.CDLL(build_oracle())
        vp, ip, fp, dp = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_double)
        L.orc_create.restype = vp
        L.orc_create.argtypes = [C.POINTER(_Cfg), vp, vp, vp] + [C.POINTER(vp)] * 9
        L.orc_destroy.argtypes = [vp]
        L.orc_forward.restype = C.c_int
        L.orc_forward.argtypes = [vp, vp, vp, C.c_int, C.c_int, vp, vp, vp]
        L.orc_lm_head.argtypes = [vp, vp, C.c_int, vp]
        L.orc_confidence.argtypes = [vp, C.c_int, C.c_double, C.c_double, dp, dp, C.POINTER(C.c_int)]
        L.orc_rmsnorm.argtypes = [vp, vp, C.c_int, C.c_float, vp]
        L.orc_rope.argtypes = [vp, C.c_int, C.c_int, C.c_float]
        L.orc_silu.restype = C.c_double
        L.orc_silu.argtypes = [C.c_double]
        L.orc_attention_head.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, vp]
        L.orc_dot_row.restype = C.c_double
        L.orc_dot_row.argtypes = [vp, C.c_int, C.c_size_t, C.c_int, vp]
        L.orc_matmul_rows.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, C.c_int, vp]
        L.orc_round_bf16.restype = C.c_float
        L.orc_round_bf16.argtypes = [C.c_float]
        L.orc_round_fp16.restype = C.c_float
        L.orc_round_fp16.argtypes = [C.c_float]
        L.orc_fp16_bits_to_f32.restype = C.c_float
        L.orc_fp16_bits_to_f32.argtypes = [C.c_uint16]
        L.orc_read_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp]
        _LIB = L
    return _LIB


def _as_host_array(t):
    """torch tensor (cpu; bf16, fp16 or fp32) or ndarray -> contiguous ndarray viewing the storage bits (bf16 as
    uint16, fp16 as float16)."""
    if isinstance(t, np.ndarray):
        return np.ascontiguousarray(t)
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def confidence_of_logits(logits: np.ndarray, clamp: float = CLAMP, eps_h: float = EPS_H):
    """(confidence, p_max, argmax) of one fp32 logits row: Eq. 1-4 evaluated literally in double."""
    a = np.ascontiguousarray(logits, dtype=np.float32)
    conf, pm, am = C.c_double(), C.c_double(), C.c_int()
    lib().orc_confidence(_ptr(a), a.shape[0], clamp, eps_h, C.byref(conf), C.byref(pm), C.byref(am))
    return conf.value, pm.value, am.value


class OracleModel:
    """The target model (and, with a skip mask, the draft model) with its KV cache."""

    def __init__(self, shape, weights: Dict[str, object]):
        self.shape = shape
        self.L, self.d, self.V = shape.n_layers, shape.d_model, shape.vocab
        self._keep = {}
        wd = {"fp32": 0, "bf16": 1, "fp16": 2}[shape.weight_dtype]

        def hold(name, t):
            a = _as_host_array(t)
            exp = np.float32 if (wd == 0 or name.startswith(("norm", "final"))) else (np.uint16 if wd == 1 else np.float16)
            assert a.dtype == exp, (name, a.dtype)
            self._keep[name] = a
            return _ptr(a)

        def ptr_list(name):
            arr = (C.c_void_p * self.L)(*[hold(f"{name}{l}", weights[name][l]) for l in range(self.L)])
            self._keep["p_" + name] = arr
            return arr

        cfg = _Cfg(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                   shape.max_seq, shape.rms_eps, shape.rope_theta, wd, getattr(shape, "kv_heads", shape.n_heads))
        lists = [ptr_list(n) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")]
        self._h = lib().orc_create(C.byref(cfg), hold("embed", weights["embed"]), hold("lm_head", weights["lm_head"]),
                                   hold("final_norm", weights["final_norm"]), *lists)
        if not self._h:
            raise MemoryError("orc_create failed")

    def close(self):
        if getattr(self, "_h", None):
            lib().orc_destroy(self._h)
            self._h = None

    __del__ = close

    def forward(self, tokens, pos0: int, skip_mask: Optional[np.ndarray] = None, want_logits: bool = True,
                want_hidden: bool = False):
        """Run ``tokens`` at positions pos0.. through the kept layers; returns dict with
        logits [n,V] (fp32) and, if asked, hid_attn / hid_ffn [L,n,d]."""
        tok = np.ascontiguousarray(tokens, dtype=np.int32)
        n = tok.shape[0]
        logits = np.empty((n, self.V), np.float32) if want_logits else None
        ha = np.empty((self.L, n, self.d), np.float32) if want_hidden else None
        hf = np.empty((self.L, n, self.d), np.float32) if want_hidden else None
        mask = None if skip_mask is None else np.ascontiguousarray(skip_mask, dtype=np.uint8)
        rc = lib().orc_forward(self._h, None if mask is None else _ptr(mask), _ptr(tok), n, int(pos0),
                               None if logits is None else _ptr(logits),
                               None if ha is None else _ptr(ha), None if hf is None else _ptr(hf))
        if rc != 0:
            raise ValueError("orc_forward: bad argument (token id or position out of range)")
        return {"logits": logits, "hid_attn": ha, "hid_ffn": hf}

    def lm_head(self, hidden: np.ndarray) -> np.ndarray:
        """Final RMSNorm + shared LM head on hidden rows [n,d] -> logits [n,V]."""
        h = np.ascontiguousarray(hidden, dtype=np.float32)
        out = np.empty((h.shape[0], self.V), np.float32)
        lib().orc_lm_head(self._h, _ptr(h), h.shape[0], _ptr(out))
        return out

    def read_kv(self, layer: int, which: int, pos: int) -> np.ndarray:
        out = np.empty(getattr(self.shape, "kv_heads", self.shape.n_heads) * self.shape.head_dim, np.float32)
        lib().orc_read_kv(self._h, layer, which, pos, _ptr(out))
        return out
