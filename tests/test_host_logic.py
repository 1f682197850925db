"""Host-side checks that need no GPU: the C-ABI library loads, exports every declared
symbol, validates arguments before touching the device, and its layout helpers agree with
the oracle's independent statement of the 128x4 scale layout."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mxfp8.h")).read()
    body = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mxfp8_[a-z0-9_]+)\s*\(", body))
    assert declared, "no declarations found"
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(B.EXPORTS)
    for name in B.EXPORTS:
        assert name in declared, name


def test_scale_bytes_and_offsets_match_oracle_layout():
    for rows, cols in ((256, 512), (96, 8288), (32, 32), (1000, 4096)):
        for o, mn, nkb in ((B.ROW, rows, cols // 32), (B.COL, cols, rows // 32)):
            if nkb == 0:
                continue
            assert B.mxfp8_scale_bytes(rows, cols, o, B.SF_LINEAR) == mn * nkb
            assert B.mxfp8_scale_bytes(rows, cols, o, B.SF_SWIZZLED) == ((mn + 127) // 128) * ((nkb + 3) // 4) * 512
            rng = np.random.default_rng(rows + cols)
            for _ in range(200):
                m, k = int(rng.integers(mn)), int(rng.integers(nkb))
                assert B.mxfp8_sf_offset(m, k, nkb, B.SF_SWIZZLED) == orc.sf_offset_swizzled(m, k, nkb)
                assert B.mxfp8_sf_offset(m, k, nkb, B.SF_LINEAR) == m * nkb + k
    assert B.mxfp8_sf_offset(0, 5, 4, B.SF_SWIZZLED) == -1


def test_argument_validation_happens_on_the_host():
    L = B.lib()
    p = ctypes.c_void_p(0x1000)  # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1004)
    q = L.mxfp8_quantize
    assert q(None, B.BF16, 32, 32, B.ROW, 0, 0, p, p, None, None, 0, None) == -1
    assert q(p, 7, 32, 32, B.ROW, 0, 0, p, p, None, None, 0, None) == -2
    assert q(p, B.BF16, 32, 32, 0, 0, 0, p, p, None, None, 0, None) == -2
    assert q(p, B.BF16, 32, 32, B.ROW, 2, 0, p, p, None, None, 0, None) == -2
    assert q(p, B.BF16, 32, 32, B.ROW, 0, 2, p, p, None, None, 0, None) == -2
    assert q(p, B.BF16, 32, 32, B.ROW, 0, 0, p, p, None, None, 5, None) == -2
    assert q(p, B.BF16, 32, 32, B.BOTH, 0, 0, p, p, None, p, 0, None) == -1
    assert q(p, B.BF16, 0, 32, B.ROW, 0, 0, p, p, None, None, 0, None) == -3
    assert q(p, B.BF16, 32, 48, B.ROW, 0, 0, p, p, None, None, 0, None) == -3
    assert q(p, B.BF16, 48, 32, B.COL, 0, 0, None, None, p, p, 0, None) == -3
    assert q(odd, B.BF16, 32, 32, B.ROW, 0, 0, p, p, None, None, 0, None) == -4
    assert q(p, B.BF16, 32, 32, B.ROW, 0, 0, odd, p, None, None, 0, None) == -4
    d = L.mxfp8_dequantize
    assert d(p, p, 32, 32, B.BOTH, 0, 0, p, 0, None) == -2
    assert d(p, None, 32, 32, B.ROW, 0, 0, p, 0, None) == -1
    assert d(p, p, 32, 40, B.ROW, 0, 0, p, 0, None) == -3
    g = L.mxfp8_gemm
    assert g(None, p, p, p, 128, 128, 128, 0, 0, 0, 0, p, 0, None, None, 0, None) == -1
    assert g(p, p, p, p, 128, 128, 100, 0, 0, 0, 0, p, 0, None, None, 0, None) == -3
    assert g(p, p, p, p, 128, 128, 128, 3, 0, 0, 0, p, 0, None, None, 0, None) == -2
    assert g(p, p, p, p, 100, 128, 128, 1, 0, 0, 0, p, 0, None, None, 0, None) == -5   # MN-major A needs M % 16 == 0
    assert g(p, p, p, p, 128, 130, 128, 0, 0, 0, 0, p, 1, None, None, 0, None) == -5   # BF16 output needs N % 8 == 0
    assert "timeout" in B.status_string(-7) or "wait" in B.status_string(-7)
