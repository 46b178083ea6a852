"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header declares, and
rejects bad configurations before touching CUDA."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2503_01330_b200 import binding
from paper_2503_01330_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "wkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wkv_[a-z_]+)\s*\(", text)) - {"wkv_alloc_fn", "wkv_release_fn"})


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), f"libwkv.so does not export {n}"
    assert sorted(binding.EXPORTS) == names           # the binding lists exactly the header's functions


def test_error_texts(lib):
    for code in range(0, -6, -1):
        assert lib.wkv_strerror(code).decode() != "unknown error"
    assert lib.wkv_strerror(-99).decode() == "unknown error"


GOOD = dict(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=4, head_dim=64, budget=128, window=16, sink=0,
            dtype=binding.WKV_F32, scale=0.0, merge=1, n_splits=0)


@pytest.mark.parametrize("change,fragment", [
    ({}, None),
    ({"window": 0}, "window"),
    ({"sink": -1}, "sink"),
    ({"budget": 10, "window": 8, "sink": 4}, "sink + window"),
    ({"budget": 0}, "budget"),
    ({"budget": 1 << 20}, "budget"),
    ({"head_dim": 96}, "head_dim"),
    ({"n_q_heads": 6, "n_kv_heads": 4}, "multiple"),
    ({"n_q_heads": 12, "n_kv_heads": 4}, "1, 2, 4 or 8"),
    ({"dtype": 7}, "dtype"),
    ({"merge": 2}, "merge"),
    ({"n_splits": 65}, "n_splits"),
    ({"scale": -1.0}, "scale"),
    ({"n_layers": 0}, "n_layers"),
    ({"schedule": 4}, "schedule"),
])
def test_config_validation(lib, change, fragment):
    cfg = binding.make_config(**{**GOOD, **change})
    msg = binding.wkv_config_error(cfg)
    if fragment is None:
        assert msg is None
    else:
        assert msg is not None and fragment in msg
        h = C.c_void_p()
        assert lib.wkv_create(C.byref(cfg), C.byref(h)) == binding.WKV_ERR_INVALID and not h.value


def test_null_arguments(lib):
    assert lib.wkv_create(None, None) == binding.WKV_ERR_INVALID
    h = C.c_void_p()
    assert lib.wkv_create(None, C.byref(h)) == binding.WKV_ERR_INVALID
    assert lib.wkv_decode_step(None, 0, None, None, None, None, None, None) == binding.WKV_ERR_INVALID
    assert lib.wkv_status(None) == binding.WKV_ERR_INVALID
    lib.wkv_destroy(None)
    assert lib.wkv_launch_count(None) == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_create_without_gpu_fails_loudly(lib):
    cfg = binding.make_config(**GOOD)
    h = C.c_void_p()
    assert lib.wkv_create(C.byref(cfg), C.byref(h)) == binding.WKV_ERR_CUDA and not h.value
    with pytest.raises(Exception):
        binding.Context(1, 1, 4, 4, 64, 128, 16, dtype=binding.WKV_F32)
