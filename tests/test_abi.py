"""The shared library builds, loads and exports every entry point the header declares; host-side
argument checks answer without touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2407_12021_b200 import build
    build.build()
    from paper_2407_12021_b200 import binding
    return binding


def _declared():
    text = open(os.path.join(ROOT, "include", "aded.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aded_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "aded_verify" in names and "aded_trigram_update" in names and "aded_trigram_topk" in names
    cdll = ctypes.CDLL(os.path.join(ROOT, "paper_2407_12021_b200", "libaded.so"))
    for n in names:
        assert hasattr(cdll, n), n
    assert sorted(lib.EXPORTS) == names


def test_status_strings(lib):
    assert lib.aded_status_string(0) == "ok"
    assert "tree" in lib.aded_status_string(2)
    assert lib.aded_status_string(99) == "unknown status"


def test_null_and_range_checks_do_not_need_a_device(lib):
    L = lib._lib
    out = ctypes.c_void_p()
    assert L.aded_model_create(None, None, ctypes.byref(out)) == 1
    assert L.aded_model_destroy(None) == 1
    assert L.aded_kv_create(None, 1, None, ctypes.byref(out)) == 1
    assert L.aded_verify(None, None, None, None, 4, None, None, None) == 1
    assert L.aded_trigram_create(None, ctypes.byref(out)) == 1
    cfg = lib.TrigramConfig(100, 2, 0, 0, 0)          # too few buckets
    assert L.aded_trigram_create(ctypes.byref(cfg), ctypes.byref(out)) == 1
    assert L.aded_trigram_update(None, None, 5, None) == 1
    assert L.aded_trigram_topk(None, None, 1, 4, None, None, None, None) == 1
    mc = lib.ModelConfig(1, 100, 1, 100, 64, 10, 0, 1e-5, 1e4, 4, 1)   # head_dim 100 is not covered
    w = lib.Weights(1, 1, 1, (lib.LayerWeights * 1)(lib.LayerWeights(1, 1, 1, 1, 1, 1)))
    assert L.aded_model_create(ctypes.byref(mc), ctypes.byref(w), ctypes.byref(out)) == 7
    mc = lib.ModelConfig(1, 128, 2, 64, 64, 10, 5, 1e-5, 1e4, 4, 1)    # unknown dtype
    assert L.aded_model_create(ctypes.byref(mc), ctypes.byref(w), ctypes.byref(out)) == 1
