"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and
rejects host-detectable errors before touching the device."""
import ctypes as C
import os
import re

import pytest

import paper_2511_07427_b200 as P
from paper_2511_07427_b200.binding import _Config

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names |= set(re.findall(r"\b(dynakv_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    L = P.load_library()
    declared = _declared_symbols()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} is declared in include/ but not exported"
    assert set(P.EXPORTED_SYMBOLS) <= declared


def _cfg(**kw):
    base = dict(n_units=1, gqa_group=4, head_dim=64, kv_dtype=0, max_tokens=128, max_clusters=16, kmeans_iters=2,
                init_mode=0, split_size_factor=2.0, split_var_factor=2.0, split_min_size=8, split_iters=8, trace=0,
                assign_mode=0, attn_mode=0)
    base.update(kw)
    return _Config(**base)


@pytest.mark.parametrize("bad", [dict(n_units=0), dict(gqa_group=0), dict(gqa_group=9), dict(head_dim=96),
                                 dict(kv_dtype=3), dict(kv_dtype=2, head_dim=64), dict(max_tokens=0), dict(max_clusters=0), dict(max_clusters=5000),
                                 dict(kmeans_iters=0), dict(split_iters=0), dict(init_mode=2),
                                 dict(update_mode=4), dict(update_mode=-1), dict(update_mode=2, local_max=1),
                                 dict(update_mode=3, buf_max=0)])
def test_create_rejects_bad_config_without_a_device(bad):
    L = P.load_library()
    h = C.c_void_p()
    c = _cfg(**bad)
    assert L.dynakv_create(C.byref(c), None, C.byref(h)) == -1
    assert not h.value


def test_null_arguments_are_rejected():
    L = P.load_library()
    h = C.c_void_p()
    assert L.dynakv_create(None, None, C.byref(h)) == -1
    assert L.dynakv_create(C.byref(_cfg()), None, None) == -1
    assert L.dynakv_build_index(None, None, None, 0, 64, 1, 0) == -1
    assert L.dynakv_append(None, None, None) == -1
    assert L.dynakv_decode_step(None, None, 1, None, None) == -1
    assert L.dynakv_split_check(None) == -1
    assert L.dynakv_decode_loop(None, None, None, None, 0, 1, None) == -1
    assert L.dynakv_step_host(None, None, None, None, 1, None) == -1
    assert L.dynakv_get_status(None, None) == -1
    assert L.dynakv_export_state(None, None, None, None, None, None, None, None) == -1
    assert L.dynakv_launch_count(None) == 0
    L.dynakv_destroy(None)


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(P.DynaKVError):
        P.DynaKV(P.DynaKVConfig(n_units=1, gqa_group=1, head_dim=64, kv_dtype=P.F32, max_tokens=64, max_clusters=4))
