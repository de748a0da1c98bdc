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
    assert mb.morello_select_path(1, 16, 100, 100) == mb.MORELLO_PATH_SKINNY       # ... one chunk of rows: not worth copying
    assert mb.morello_select_path(1, 17, 100, 100) == mb.MORELLO_PATH_TCGEN05      # ... two chunks: padded copies are cheaper
    assert mb.morello_select_path(1, 4096, 4096, 4095) == mb.MORELLO_PATH_TCGEN05  # ... through zero-padded copies
    assert mb.morello_select_path(1, 512, 1001, 1000) == mb.MORELLO_PATH_TCGEN05   # k % 8 != 0 likewise
    assert mb.morello_select_path(1, 4096, 4096, 4096) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(8, 2048, 2048, 16384) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(1, 17, 8, 8) == mb.MORELLO_PATH_TCGEN05
    assert mb.morello_select_path(1, -1, 4, 4) == -1


def test_route_description_names_the_kernel(mb):
    d = mb.morello_describe_route
    assert d(1, 1, 2048, 16384).startswith("fma gemv_stream_kernel")          # the headline GEMV
    assert "256 strips" in d(1, 1, 2048, 16384)
    assert d(1, 16, 2048, 16384).startswith("tcgen05 swap_kernel")            # operands swapped
    assert "16 rows" in d(1, 16, 2048, 16384)
    assert "a CTA pair per 256 x 256 tile" in d(1, 4096, 4096, 4096)
    assert "one CTA per 128 x" in d(1, 128, 2048, 16384)
    assert "k slices through the workspace" in d(1, 512, 16384, 2048)
    assert "added inside a cluster" in d(1, 16, 16384, 2048)
    assert d(1, 2048, 2047, 2049).startswith("padded copies of A B to k=2048 n=2056 (C written from registers), then tcgen05")
    assert d(1, 512, 1001, 1000).startswith("padded copies of A B to k=1008 n=1000, then tcgen05")
    assert d(1, 4, 4, 16).startswith("fma skinny_kernel")
    assert "shifted columns" in d(1, 1, 2048, 16383)
    assert d(0, 4, 4, 4).startswith("nothing to launch")
    # a short buffer is filled up to its last byte and NUL-terminated; bad arguments are refused
    buf = ctypes.create_string_buffer(b"x" * 12, 12)
    assert mb.lib().morello_describe_route(1, 4096, 4096, 4096, buf, 12) == mb.MORELLO_OK
    assert buf.raw == b"tcgen05 gem\0"
    assert mb.lib().morello_describe_route(1, 4, 4, 4, None, 0) == mb.MORELLO_ERR_NULL_POINTER
    assert mb.lib().morello_describe_route(1, -4, 4, 4, buf, 12) == mb.MORELLO_ERR_INVALID_SHAPE


def test_per_device_setup_runs_once_per_device_and_retries_failures(mb):
    once = mb.morello_selftest_per_device_once
    assert once(1, 5) == 1          # one device, five calls: set up once
    assert once(4, 3) == 5          # four devices: once each, plus device 1's failed first attempt
    assert once(4, 1) == 4
    assert once(0, 3) == 0
    assert once(-1, 3) == -1


def test_missing_library_fails_loudly(mb, monkeypatch):
    import importlib
    from paper_2505_01637_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libmorello.so"))
    with pytest.raises(ImportError):
        binding.morello_version()
    monkeypatch.undo()
    importlib.reload(binding)
