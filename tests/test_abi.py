"""The C boundary without a GPU: the library loads and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2406_07368_b200 import build
    return build.build()


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(la_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(built):
    L = ctypes.CDLL(built)
    declared = _declared()
    assert {"la_create", "la_destroy", "la_prefill", "la_decode_step", "la_verify_tree", "la_commit"} <= declared
    for name in declared:
        assert hasattr(L, name), f"{name} is declared in include/ but not exported"
    from paper_2406_07368_b200 import binding
    assert set(binding.EXPORTS) == declared


def test_host_side_rejections_need_no_gpu(built):
    from paper_2406_07368_b200 import binding
    L = binding.lib()
    assert L.la_status_str(0) == b"LA_OK" and L.la_status_str(4) == b"LA_ERR_BAD_TREE"
    h = ctypes.c_void_p()
    bad = binding.la_config(32, 96, 3, 0, 0, 0.0, 1, 64, 8)          # unsupported head dimension
    assert L.la_create(ctypes.byref(bad), ctypes.byref(h)) == binding.LA_ERR_UNSUPPORTED
    bad = binding.la_config(32, 128, 33, 0, 0, 0.0, 1, 64, 8)         # too many taps
    assert L.la_create(ctypes.byref(bad), ctypes.byref(h)) == binding.LA_ERR_INVALID_ARG
    bad = binding.la_config(32, 128, 3, 0, 0, 0.0, 1, 65, 8)          # too many nodes
    assert L.la_create(ctypes.byref(bad), ctypes.byref(h)) == binding.LA_ERR_INVALID_ARG
    assert L.la_create(None, ctypes.byref(h)) == binding.LA_ERR_INVALID_ARG
    st = binding.la_state(None, None, None, None)
    assert L.la_prefill(None, 1, 1, None, None, None, None, 0, ctypes.byref(st), None, None) == binding.LA_ERR_INVALID_ARG
    assert L.la_decode_step(None, 1, None, None, None, None, ctypes.byref(st), None, None) == binding.LA_ERR_INVALID_ARG
    assert L.la_destroy(None) == binding.LA_ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2406_07368_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libla_b200.so")
    with pytest.raises(RuntimeError, match="no CPU or eager fallback"):
        binding.lib()
