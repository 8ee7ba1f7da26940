"""ctypes binding of libconflayers.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
import re
from typing import Dict, List, Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libconflayers.so")
_HEADER = os.path.join(os.path.dirname(_PKG), "include", "conflayers.h")
CL_MAX_K = 8
_ERRNAMES = {0: "CL_OK", 1: "CL_EINVAL", 2: "CL_ENOMEM", 3: "CL_ECUDA", 4: "CL_ESTATE", 5: "CL_ERANGE", 6: "CL_ETIMEOUT"}


class ConfLayersError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{_ERRNAMES.get(code, code)}: {msg}")
        self.code = code


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab",
                                       "max_seq")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("weight_dtype", C.c_int), ("tap_positions", C.c_int),
                ("tap_modules", C.c_int)]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")] + \
               [("on_device", C.c_int), ("head_only", C.c_int)]


class SelectCfg(C.Structure):
    _fields_ = [("w_base", C.c_double), ("lam", C.c_double), ("eps", C.c_double), ("flat_tol", C.c_double),
                ("w_max", C.c_double), ("lo", C.c_int), ("hi", C.c_int), ("n_skip", C.c_int),
                ("min_ratio", C.c_double), ("fixed_window", C.c_int)]

    @classmethod
    def make(cls, lo: int, hi: int, n_skip: int = -1, w_base: float = 2.0, lam: float = 0.3, eps: float = 1e-8,
             flat_tol: float = 1e-3, w_max: float = 0.0, min_ratio: float = 0.4, fixed_window: int = 0) -> "SelectCfg":
        return cls(w_base, lam, eps, flat_tol, w_max, lo, hi, n_skip, min_ratio, fixed_window)


CL_MAX_ROUNDS = 32
CL_DEBUG_WAIT_LIMIT_US, CL_DEBUG_BARRIER_EXTRA, CL_DEBUG_DEVICE_ERR = 1, 2, 3


class SearchCfg(C.Structure):
    _fields_ = [("K", C.c_int), ("interval", C.c_int), ("max_rounds", C.c_int), ("score_goal", C.c_float)]


class SearchReport(C.Structure):
    _fields_ = [("n_scored", C.c_int), ("best_round", C.c_int), ("searching", C.c_int),
                ("scores", C.c_float * (CL_MAX_ROUNDS + 1))]


class Stats(C.Structure):
    _fields_ = [("cycles", C.c_uint64), ("drafted", C.c_uint64), ("accepted", C.c_uint64), ("emitted", C.c_uint64),
                ("ctx_len", C.c_int), ("n_skipped", C.c_int), ("kernel_launches", C.c_uint64)]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def exported_symbols() -> List[str]:
    """Function names declared in include/conflayers.h."""
    src = open(_HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(cl_[a-z_]+)\s*\(", src)))


def load_library():
    """dlopen the in-tree library (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(f"{_LIB_PATH} not built; run `python -m paper_2604_14612_b200.build` "
                                "(or __graft_entry__.build())")
    L = C.CDLL(_LIB_PATH)
    vp, ip, fp = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float)
    sig = {
        "cl_create": [C.POINTER(ModelCfg), vp, C.POINTER(vp)],
        "cl_load": [vp, C.POINTER(Weights)],
        "cl_destroy": [vp],
        "cl_prefill": [vp, vp, C.c_int, C.c_int, ip],
        "cl_set_skip_set": [vp, vp],
        "cl_get_skip_set": [vp, vp],
        "cl_draft": [vp, C.c_int, C.c_float, vp, vp, vp, vp, C.POINTER(C.c_int)],
        "cl_verify": [vp, C.c_int, vp, vp],
        "cl_accept": [vp, C.POINTER(C.c_int), vp],
        "cl_step_vanilla": [vp, ip],
        "cl_generate": [vp, C.c_int, C.c_int, vp, C.POINTER(C.c_int), C.POINTER(Stats)],
        "cl_generate_search": [vp, C.POINTER(SearchCfg), C.POINTER(SelectCfg), C.c_int, vp, C.POINTER(C.c_int),
                               C.POINTER(SearchReport), vp],
        "cl_rollback": [vp, C.c_int, C.c_int32],
        "cl_force_tokens": [vp, vp, C.c_int],
        "cl_layer_confidences": [vp, vp, C.c_int, C.c_int, vp, vp, vp, vp],
        "cl_select_skip_set": [vp, C.POINTER(SelectCfg), vp, vp, vp],
        "cl_score_loop": [vp, C.POINTER(SelectCfg), C.POINTER(vp), C.c_int, C.c_int, vp, vp, C.POINTER(C.c_int), vp, vp],
        "cl_read_hidden_ring": [vp, vp],
        "cl_get_stats": [vp, C.POINTER(Stats)],
        "cl_debug_set": [vp, C.c_int, C.c_longlong],
        "cl_debug_read": [vp, C.c_int, vp, C.c_int],
        "cl_layer_confidences_static": [vp, vp, C.c_int, C.c_int, C.c_int, C.c_float, vp, C.c_int, vp, vp, vp, vp],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = C.c_int
    L.cl_last_error.argtypes = [vp]
    L.cl_last_error.restype = C.c_char_p
    _lib = L
    return L


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def cl_layer_confidences_static(lm_head, final_norm, hidden, rms_eps: float = 1e-5, stream: Optional[int] = None):
    """Context-free confidence scoring that allocates no device memory (see the header for who needs it).

    lm_head [V, d], hidden [..., d] (same dtype, bf16 or fp32) and final_norm fp32 [d] are CUDA tensors;
    returns dict(conf, p_max, argmax) as numpy arrays with hidden's leading shape."""
    L = load_library()
    import torch
    if not (lm_head.is_cuda and hidden.is_cuda and final_norm.is_cuda):
        raise ValueError("lm_head, hidden and final_norm must be CUDA tensors")
    if not (lm_head.is_contiguous() and hidden.is_contiguous() and final_norm.is_contiguous()):
        raise ValueError("lm_head, hidden and final_norm must be contiguous")
    dtypes = {torch.float32: 0, torch.bfloat16: 1}          # the storage types the call supports
    if lm_head.dtype not in dtypes:
        raise ValueError(f"lm_head dtype {lm_head.dtype} not supported: float32 or bfloat16 only")
    if hidden.dtype != lm_head.dtype or final_norm.dtype != torch.float32:
        raise ValueError("hidden must have lm_head's dtype and final_norm must be float32")
    if lm_head.dim() != 2 or hidden.dim() < 1:
        raise ValueError("lm_head must be [vocab, d_model] and hidden [..., d_model]")
    V, d = lm_head.shape
    if hidden.shape[-1] != d or tuple(final_norm.shape) != (d,):
        raise ValueError(f"hidden's last dimension and final_norm must have d_model = {d} elements")
    lead = tuple(hidden.shape[:-1])
    n = int(np.prod(lead))
    conf = np.zeros(n, np.float32)
    pm = np.zeros(n, np.float32)
    am = np.zeros(n, np.int32)
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    rc = L.cl_layer_confidences_static(lm_head.data_ptr(), final_norm.data_ptr(), V, d,
                                       dtypes[lm_head.dtype], rms_eps, hidden.data_ptr(), n,
                                       C.c_void_p(stream), _np_ptr(conf), _np_ptr(pm), _np_ptr(am))
    if rc:
        raise ConfLayersError(rc, L.cl_last_error(None).decode())
    return dict(conf=conf.reshape(lead), p_max=pm.reshape(lead), argmax=am.reshape(lead))


class Context:
    """One model on one CUDA stream.  Methods mirror the C calls and return numpy values."""

    def __init__(self, n_layers: int, d_model: int, n_heads: int, d_ffn: int, vocab: int, max_seq: int,
                 weight_dtype: str = "bf16", rms_eps: float = 1e-5, rope_theta: float = 10000.0,
                 tap_positions: int = 0, stream: Optional[int] = None, n_kv_heads: int = 0, tap_modules: int = 1):
        self._L = load_library()
        self.cfg = ModelCfg(n_layers, d_model, n_heads, n_kv_heads or n_heads, d_model // n_heads, d_ffn, vocab, max_seq, rms_eps,
                            rope_theta, {"fp32": 0, "bf16": 1, "fp16": 2}[weight_dtype], tap_positions, tap_modules)
        self.taps = 2 if tap_modules == 2 else 1
        self.weight_dtype = weight_dtype
        self._h = C.c_void_p()
        if stream is None:
            import torch
            stream = torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0
        rc = self._L.cl_create(C.byref(self.cfg), C.c_void_p(stream), C.byref(self._h))
        if rc:
            raise ConfLayersError(rc, self._L.cl_last_error(None).decode())

    @classmethod
    def from_shape(cls, shape, tap_positions: int = 0, stream: Optional[int] = None, tap_modules: int = 1) -> "Context":
        return cls(shape.n_layers, shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab, shape.max_seq,
                   shape.weight_dtype, shape.rms_eps, shape.rope_theta, tap_positions, stream,
                   getattr(shape, "kv_heads", shape.n_heads), tap_modules)

    # -- helpers
    def _ck(self, rc: int):
        if rc:
            raise ConfLayersError(rc, self._L.cl_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            self._L.cl_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- life cycle
    def cl_load(self, weights: Dict[str, object], head_only: bool = False):
        """weights: dict of torch tensors as made by ``synth.make_weights`` (on the CUDA device or on the host)."""
        L = self.cfg.n_layers
        keep = []

        def ptr(t):
            t = t.contiguous()
            keep.append(t)
            return t.data_ptr()

        on_dev = bool(weights["lm_head"].is_cuda)
        w = Weights()
        w.lm_head = ptr(weights["lm_head"])
        w.final_norm = ptr(weights["final_norm"].float())
        w.on_device = 1 if on_dev else 0
        w.head_only = 1 if head_only else 0
        if not head_only:
            w.embed = ptr(weights["embed"])
            for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2"):
                arr = (C.c_void_p * L)(*[ptr(weights[n][l].float() if n.startswith("norm") else weights[n][l])
                                         for l in range(L)])
                keep.append(arr)
                setattr(w, n, arr)
        self._ck(self._L.cl_load(self._h, C.byref(w)))

    def cl_prefill(self, tokens: Sequence[int], tap_hidden: bool = False) -> int:
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        first = C.c_int32()
        self._ck(self._L.cl_prefill(self._h, _np_ptr(t), t.shape[0], int(tap_hidden), C.byref(first)))
        return first.value

    def cl_set_skip_set(self, mask: Sequence[int]):
        m = np.ascontiguousarray(mask, dtype=np.uint8)
        assert m.shape[0] == self.cfg.n_layers
        self._ck(self._L.cl_set_skip_set(self._h, _np_ptr(m)))

    def cl_get_skip_set(self) -> np.ndarray:
        m = np.zeros(self.cfg.n_layers, np.uint8)
        self._ck(self._L.cl_get_skip_set(self._h, _np_ptr(m)))
        return m

    def cl_draft(self, K: int, stop_p: float = 0.0, want_logits: bool = False):
        toks = np.zeros(CL_MAX_K, np.int32)
        pm = np.zeros(CL_MAX_K, np.float32)
        cf = np.zeros(CL_MAX_K, np.float32)
        lg = np.zeros((max(K, 1), self.cfg.vocab), np.float32) if want_logits else None
        n = C.c_int()
        self._ck(self._L.cl_draft(self._h, K, stop_p, _np_ptr(toks), _np_ptr(pm), _np_ptr(cf), _np_ptr(lg), C.byref(n)))
        k = n.value
        return dict(tokens=toks[:k].copy(), p_max=pm[:k].copy(), conf=cf[:k].copy(),
                    logits=None if lg is None else lg[:k], n_drafted=k)

    def cl_force_tokens(self, toks: Sequence[int]):
        t = np.ascontiguousarray(toks, dtype=np.int32)
        self._ck(self._L.cl_force_tokens(self._h, _np_ptr(t), t.shape[0]))

    def cl_verify(self, n_rows: int, tap_hidden: bool = False, want_logits: bool = False):
        """n_rows = drafted + 1 (only used to size the outputs)."""
        tg = np.zeros(CL_MAX_K + 1, np.int32)
        lg = np.zeros((n_rows, self.cfg.vocab), np.float32) if want_logits else None
        self._ck(self._L.cl_verify(self._h, int(tap_hidden), _np_ptr(tg), _np_ptr(lg)))
        return dict(targets=tg[:n_rows].copy(), logits=lg)

    def cl_accept(self):
        n = C.c_int()
        em = np.zeros(CL_MAX_K + 1, np.int32)
        self._ck(self._L.cl_accept(self._h, C.byref(n), _np_ptr(em)))
        return n.value, em[:n.value + 1].copy()

    def cl_step_vanilla(self) -> int:
        t = C.c_int32()
        self._ck(self._L.cl_step_vanilla(self._h, C.byref(t)))
        return t.value

    def cl_generate(self, K: int, max_new: int):
        out = np.zeros(max_new, np.int32)
        n = C.c_int()
        st = Stats()
        self._ck(self._L.cl_generate(self._h, K, max_new, _np_ptr(out), C.byref(n), C.byref(st)))
        return out[:n.value], st

    def cl_generate_search(self, K: int, max_new: int, interval: int, score_goal: float, max_rounds: int, sel: SelectCfg):
        out = np.zeros(max_new, np.int32)
        n = C.c_int()
        rep = SearchReport()
        L = self.cfg.n_layers
        masks = np.zeros((max_rounds + 1, L), np.uint8)
        cfg = SearchCfg(K, interval, max_rounds, score_goal)
        self._ck(self._L.cl_generate_search(self._h, C.byref(cfg), C.byref(sel), max_new, _np_ptr(out), C.byref(n),
                                            C.byref(rep), _np_ptr(masks)))
        k = rep.n_scored
        return dict(tokens=out[:n.value], scores=[float(rep.scores[i]) for i in range(k)],
                    sets=[[l for l in range(L) if masks[i][l]] for i in range(k)], best_round=rep.best_round,
                    searching=bool(rep.searching), final_set=[l for l in range(L) if self.cl_get_skip_set()[l]])

    def cl_rollback(self, ctx_len: int, pending_token: int):
        self._ck(self._L.cl_rollback(self._h, ctx_len, pending_token))

    def cl_layer_confidences(self, hidden=None, rows: int = 0, P: int = 0):
        """hidden: CUDA tensor [rows, P, d] in the storage type, or None for the context's ring."""
        if hidden is None:
            rows, P = self.cfg.n_layers, self.taps * self.cfg.tap_positions
            hp = None
        else:
            assert hidden.is_cuda and hidden.is_contiguous()
            rows, P = hidden.shape[0], hidden.shape[1]
            hp = hidden.data_ptr()
        conf = np.zeros((rows, P), np.float32)
        pm = np.zeros((rows, P), np.float32)
        am = np.zeros((rows, P), np.int32)
        cl = np.zeros(rows, np.float32)
        self._ck(self._L.cl_layer_confidences(self._h, hp, rows, P, _np_ptr(conf), _np_ptr(pm), _np_ptr(am), _np_ptr(cl)))
        return dict(conf=conf, p_max=pm, argmax=am, c_layer=cl)

    def cl_select_skip_set(self, cfg: SelectCfg, c_layer: Optional[Sequence[float]] = None):
        L = self.cfg.n_layers
        mask = np.zeros(L, np.uint8)
        marg = np.zeros(L, np.float64)
        cl = None if c_layer is None else np.ascontiguousarray(c_layer, dtype=np.float32)
        self._ck(self._L.cl_select_skip_set(self._h, C.byref(cfg), _np_ptr(cl), _np_ptr(mask), _np_ptr(marg)))
        return mask, marg

    def cl_score_loop(self, cfg: SelectCfg, hidden_iters, scores: Sequence[float]):
        iters = len(hidden_iters)
        L = self.cfg.n_layers
        P = hidden_iters[0].shape[1]
        for h in hidden_iters:
            assert h.is_cuda and h.is_contiguous() and h.shape[0] == L and h.shape[1] == P
        ptrs = (C.c_void_p * iters)(*[h.data_ptr() for h in hidden_iters])
        sc = np.ascontiguousarray(scores, dtype=np.float32)
        best_mask = np.zeros(L, np.uint8)
        best = C.c_int()
        masks = np.zeros((iters, L), np.uint8)
        cls = np.zeros((iters, L), np.float32)
        self._ck(self._L.cl_score_loop(self._h, C.byref(cfg), ptrs, iters, P, _np_ptr(sc), _np_ptr(best_mask),
                                       C.byref(best), _np_ptr(masks), _np_ptr(cls)))
        return dict(best_mask=best_mask, best_iter=best.value, masks=masks, c_layers=cls)

    def cl_read_hidden_ring(self):
        import torch
        L, P, d = self.cfg.n_layers, self.cfg.tap_positions, self.cfg.d_model
        dt = {0: torch.float32, 1: torch.bfloat16, 2: torch.float16}[self.cfg.weight_dtype]
        out = torch.empty((L, self.taps, P, d), dtype=dt)
        self._ck(self._L.cl_read_hidden_ring(self._h, out.data_ptr()))
        return out if self.taps == 2 else out[:, 0]

    def cl_debug_set(self, what: int, value: int):
        self._ck(self._L.cl_debug_set(self._h, what, value))

    def cl_debug_read_phase_ns(self) -> np.ndarray:
        """[n_SMs, 8] nanoseconds per phase of the last persistent T-row pass (see the header)."""
        out = np.zeros((256, 8), np.uint64)
        self._ck(self._L.cl_debug_read(self._h, 1, _np_ptr(out), out.size))
        return out

    def cl_get_stats(self) -> Stats:
        st = Stats()
        self._ck(self._L.cl_get_stats(self._h, C.byref(st)))
        return st
