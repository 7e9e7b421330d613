"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names |= set(re.findall(r"SPARQ_API\s+[\w\s\*]*?\b(sparq_\w+)\s*\(", text))
    return sorted(names)


@pytest.fixture(scope="module")
def lib():
    from paper_2105_11010_b200 import build
    path = build.build_library()
    return ctypes.CDLL(path)


def test_header_declares_the_entry_points():
    names = declared_symbols()
    for must in ("sparq_quantize", "sparq_gemm_s8", "sparq_conv2d_nhwc_s8",
                 "sparq_check", "sparq_last_error", "sparq_shutdown"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_argument_validation_needs_no_gpu(lib):
    import paper_2105_11010_b200 as sparq
    from paper_2105_11010_b200._binding import _CParams
    L = sparq.load_library()
    bad = [
        _CParams(3, 4, 0x1F, 1),    # unknown mode
        _CParams(2, 5, 0x1F, 1),    # width not 2..4
        _CParams(2, 4, 0x1E, 1),    # lacks shift 0
        _CParams(2, 4, 0x0F, 1),    # lacks the top shift
        _CParams(2, 4, 0x3F, 1),    # shift above 8-n
        _CParams(2, 2, 0x41, 1),    # gap wider than the window
        _CParams(2, 4, 0x1F, 2),    # unknown rounding
    ]
    for p in bad:
        rc = L.sparq_quantize(None, None, 4, 4, ctypes.byref(p), None)
        assert rc == -1, (p.mode, p.window_bits, hex(p.placement_mask), p.rounding)
        assert sparq.sparq_last_error()
    assert L.sparq_quantize(None, None, 4, 4, None, None) == -1
    ok = _CParams(2, 4, 0x1F, 1)
    assert L.sparq_quantize(None, None, 0, 16, ctypes.byref(ok), None) == 0   # empty: no-op
    assert L.sparq_quantize(None, None, 4, 4, ctypes.byref(ok), None) == -1   # null buffers
