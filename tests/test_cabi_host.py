"""Host-only checks of the C ABI: the library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

import sb_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def binding():
    import __graft_entry__ as ge
    ge.build()
    from paper_2112_15317_b200 import binding as b
    return b


def test_library_exports_every_declared_symbol():
    b = binding()
    header = open(os.path.join(ROOT, "include", "splitbrain.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sb_[a-z_0-9]+)\s*\(", header))
    assert {"sb_model_create", "sb_forward", "sb_backward", "sb_sgd_step", "sb_loss"} <= declared
    lib = ctypes.CDLL(b.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(b.EXPORTED)


def _bytes(b, layers, **kw):
    cfg = dict(H=32, W=32, C=3, batch_per_replica=4, R=2, K=2, precision=1, flags=0)
    cfg.update(kw)
    arr = b._layers_array(layers)
    c = b.sb_config(*[cfg[k] for k in ("H", "W", "C", "batch_per_replica", "R", "K", "precision", "flags")])
    n = ctypes.c_size_t()
    return b.sb_model_bytes(arr, len(layers), ctypes.byref(c), ctypes.byref(n)), n.value


def test_model_bytes_validation():
    b = binding()
    good = si.tiny_layers()
    st, n = _bytes(b, good)
    assert st == 0 and n > 0
    assert _bytes(b, good, K=11)[0] == 2                      # K > narrowest FC width
    assert _bytes(b, good, R=0)[0] == 2
    assert _bytes(b, good, R=65)[0] == 2
    assert _bytes(b, good, precision=7)[0] == 1
    assert _bytes(b, good, H=30, W=30)[0] == 2                # 30 -> 15 -> odd at the second pool
    assert _bytes(b, good[:-1])[0] == 2                       # no loss layer
    assert _bytes(b, [(si.FC_RELU, 8), (si.CONV3X3_RELU, 8), (si.FC, 4), (si.SOFTMAX_XENT, 4)])[0] == 2
    assert _bytes(b, [(si.CONV3X3_RELU, 8), (si.FC, 4), (si.SOFTMAX_XENT, 5)])[0] == 2
    assert _bytes(b, [(9, 8), (si.FC, 4), (si.SOFTMAX_XENT, 4)])[0] == 1
    assert "unknown kind" in b.sb_last_error()
    assert b.sb_model_bytes(None, 0, None, None) == 1


def test_arena_grows_with_batch_and_shrinks_nothing_with_K():
    b = binding()
    _, n1 = _bytes(b, si.tiny_layers(), batch_per_replica=4)
    _, n2 = _bytes(b, si.tiny_layers(), batch_per_replica=8)
    assert n2 > n1


def test_create_rejects_bad_arena_without_gpu_work():
    b = binding()
    arr = b._layers_array(si.tiny_layers())
    c = b.sb_config(32, 32, 3, 4, 2, 2, 1, 0)
    h = ctypes.c_void_p()
    assert b.sb_model_create(arr, len(arr), ctypes.byref(c), None, 0, ctypes.byref(h)) == 1
    assert b.sb_model_create(arr, len(arr), ctypes.byref(c), ctypes.c_void_p(0x1001), 1 << 30, ctypes.byref(h)) == 1
    assert b.sb_model_create(arr, len(arr), ctypes.byref(c), ctypes.c_void_p(0x1000), 16, ctypes.byref(h)) == 4
