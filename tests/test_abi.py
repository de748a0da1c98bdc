"""The C-ABI library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mb():
    from paper_2505_01637_b200 import build
    build.build()
    from paper_2505_01637_b200 import binding
    binding.lib()
    return binding


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(morello_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported_and_bound(mb):
    declared = _declared_symbols()
    assert "morello_matmul_accum" in declared and len(declared) >= 12
    handle = ctypes.CDLL(mb.LIB_PATH)
    for name in declared:
        assert hasattr(handle, name), "library does not export %s" % name
        assert name in mb.SIGNATURES, "binding has no signature for %s" % name
        assert hasattr(mb, name), "binding has no wrapper for %s" % name
    assert set(mb.SIGNATURES) == declared


def test_status_strings_and_version(mb):
    assert mb.morello_status_string(mb.MORELLO_OK) == "ok"
    seen = {mb.morello_status_string(s) for s in range(0, 9)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert mb.morello_status_string(99) == "unknown status"
    assert "sm_100a" in mb.morello_version()


def test_argument_validation_needs_no_device(mb):
    L = mb.lib()
    call = L.morello_matmul_accum
    assert call(-1, 1, 1, 1, 16, 16, 16, None) == mb.MORELLO_ERR_INVALID_SHAPE
    assert call(1, 1, 1, -5, 16, 16, 16, None) == mb.MORELLO_ERR_INVALID_SHAPE
    assert call(1 << 40, 1 << 40, 1, 1, 16, 16, 16, None) == mb.MORELLO_ERR_INVALID_SHAPE
    assert call(1, 2, 3, 4, None, 16, 16, None) == mb.MORELLO_ERR_NULL_POINTER
    assert call(1, 2, 3, 4, 16, 16, None, None) == mb.MORELLO_ERR_NULL_POINTER
    assert call(1, 2, 3, 4, 17, 16, 16, None) == mb.MORELLO_ERR_MISALIGNED
    assert call(1, 2, 3, 4, 16, 16, 18, None) == mb.MORELLO_ERR_MISALIGNED
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum(1, 2, 3, 4, 0, 16, 16, 0)
    assert e.value.status == mb.MORELLO_ERR_NULL_POINTER


def test_selector_is_shape_based(mb):
    assert mb.morello_select_path(1, 1, 2048, 16384) == mb.MORELLO_PATH_SKINNY
    assert mb.morello_select_path(1, 4, 4, 16) == mb.MORELLO_PATH_SKINNY
    assert mb.morello_select_path(1, 16, 2048, 16384) == mb.MORELLO_PATH_TCGEN05   # measured crossover: 2 rows
    assert mb.morello_select_path(1, 2, 2048, 16384) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(1, 2, 2048, 1024) == mb.MORELLO_PATH_TCGEN05     # few columns: k is cut instead
    assert mb.morello_select_path(1, 16, 4096, 64) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(1, 8, 4096, 60) == mb.MORELLO_PATH_SKINNY         # n % 8 != 0: TMA cannot address it
    assert mb.morello_select_path(1, 17, 100, 100) == mb.MORELLO_PATH_SKINNY       # ... and too small to be worth copying
    assert mb.morello_select_path(1, 4096, 4096, 4095) == mb.MORELLO_PATH_TCGEN05  # ... through zero-padded copies
    assert mb.morello_select_path(1, 512, 1001, 1000) == mb.MORELLO_PATH_TCGEN05   # k % 8 != 0 likewise
    assert mb.morello_select_path(1, 4096, 4096, 4096) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(8, 2048, 2048, 16384) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(1, 17, 8, 8) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(1, -1, 4, 4) == -1


def test_missing_library_fails_loudly(mb, monkeypatch):
    import importlib
    from paper_2505_01637_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libmorello.so"))
    with pytest.raises(ImportError):
        binding.morello_version()
    monkeypatch.undo()
    importlib.reload(binding)
