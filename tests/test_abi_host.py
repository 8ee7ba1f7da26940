"""Host-side checks that need no GPU: the library builds, loads, exports every declared symbol,
and rejects bad arguments before touching a device."""
import ctypes as C

import numpy as np
import pytest

import paper_2604_14612_b200 as cl
from paper_2604_14612_b200 import build as cl_build
from paper_2604_14612_b200.binding import ModelCfg


@pytest.fixture(scope="module")
def lib():
    cl_build.build()
    return cl.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = cl.exported_symbols()
    assert len(names) >= 18 and "cl_draft" in names and "cl_layer_confidences" in names
    for n in names:
        assert hasattr(lib, n), n


def test_create_rejects_bad_shapes_before_any_device_work(lib):
    h = C.c_void_p()
    good = dict(n_layers=2, d_model=128, n_heads=2, n_kv_heads=2, head_dim=64, d_ffn=256, vocab=100, max_seq=32,
                rms_eps=1e-5, rope_theta=1e4, weight_dtype=1, tap_positions=0)
    for bad in (dict(head_dim=32, d_model=64), dict(n_kv_heads=3), dict(d_ffn=100), dict(weight_dtype=3), dict(vocab=1),
                dict(max_seq=0), dict(n_heads=3)):
        cfg = ModelCfg(**{**good, **bad})
        rc = lib.cl_create(C.byref(cfg), None, C.byref(h))
        assert rc == 1 and not h.value, bad
        assert len(lib.cl_last_error(None)) > 0
    assert lib.cl_create(None, None, C.byref(h)) == 1


def test_no_device_is_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(cl.ConfLayersError) as e:
        cl.Context(2, 128, 2, 256, 100, 32)
    assert e.value.code == 3


def test_null_context_calls_fail_cleanly(lib):
    assert lib.cl_destroy(None) == 0
    assert lib.cl_get_stats(None, None) == 1
    assert lib.cl_set_skip_set(None, None) == 1
    assert isinstance(lib.cl_last_error(None), bytes)
