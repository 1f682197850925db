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


def test_argument_validation_of_the_widened_entry_points():
    L = B.lib()
    p = ctypes.c_void_p(0x1000)          # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1004)
    # round trip
    f = L.mxfp8_fake_quantize
    assert f(None, B.BF16, 32, 32, B.ROW, 0, 0, p, None, None) == -1
    assert f(p, B.BF16, 32, 32, B.ROW, 0, 9, p, None, None) == -2
    assert f(p, B.BF16, 32, 48, B.ROW, 0, 0, p, None, None) == -3
    assert f(p, B.BF16, 32, 32, B.COL, 0, 0, p, None, None) == -1            # column output missing
    # activation / gated activation / normalisation ahead of the conversion
    a = L.mxfp8_act_quantize
    assert a(p, B.BF16, 32, 32, 9, B.ROW, 0, 0, p, p, None, None, 0, None) == -2
    assert a(p, B.BF16, 32, 32, B.ACT_RELU, B.ROW, 0, 0, p, None, None, None, 0, None) == -1
    assert a(odd, B.BF16, 32, 32, B.ACT_RELU, B.ROW, 0, 0, p, p, None, None, 0, None) == -4
    g = L.mxfp8_glu_quantize
    assert g(p, B.BF16, 32, 96, B.ACT_SILU, B.ROW, 0, 0, p, p, None, None, 0, None) == -5    # not whole 128-column tiles
    assert g(p, B.FP32, 32, 96, B.ACT_SILU, B.ROW, 0, 0, p, p, None, None, 0, None) == -5    # not whole 64-column tiles
    assert g(p, B.BF16, 32, 128, -1, B.ROW, 0, 0, p, p, None, None, 0, None) == -2
    r = L.mxfp8_rmsnorm_quantize
    assert r(p, B.BF16, 32, 32, None, 1e-5, p, B.ROW, 0, 0, p, p, None, None, 0, None) == -1
    assert r(p, B.BF16, 32, 32, p, -1.0, p, B.ROW, 0, 0, p, p, None, None, 0, None) == -3
    assert r(p, B.BF16, 32, 32, p, float("nan"), p, B.ROW, 0, 0, p, p, None, None, 0, None) == -3
    rs = L.mxfp8_rmsnorm_quantize_static
    assert rs(p, B.BF16, 65536 + 32, 32, p, 1e-5, B.ROW, 0, 0, p, p, None, None, 0, None) == -5
    # batched conversion
    items = (B._QuantizeItem * 9)()
    qm = L.mxfp8_quantize_multi
    assert qm(items, 9, B.BF16, B.ROW, 0, 0, 0, None) == -5
    assert qm(items, 0, B.BF16, B.ROW, 0, 0, 0, None) == -3
    assert qm(None, 1, B.BF16, B.ROW, 0, 0, 0, None) == -1
    assert qm(items, 1, B.BF16, B.ROW, 0, 0, 0, None) == -1                   # null source in the first item
    # several products in one launch
    probs = (B._GemmProblem * 4)()
    gm = L.mxfp8_gemm_multi
    assert gm(probs, 4, B.BF16, None) == -5
    assert gm(probs, 0, B.BF16, None) == -3
    assert gm(None, 1, B.BF16, None) == -1
    assert gm(probs, 1, 5, None) == -2
    assert gm(probs, 1, B.BF16, None) == -1                                   # null operands in the first product
    # per-expert products
    gg = L.mxfp8_grouped_gemm
    assert gg(p, p, p, p, None, 4, B.GROUP_M, 512, 128, 128, 0, 0, 0, p, 1, None) == -1
    assert gg(p, p, p, p, p, 4, 3, 512, 128, 128, 0, 0, 0, p, 1, None) == -2
    assert gg(p, p, p, p, p, 0, B.GROUP_M, 512, 128, 128, 0, 0, 0, p, 1, None) == -3
    assert gg(p, p, p, p, p, 300, B.GROUP_M, 512, 128, 128, 0, 0, 0, p, 1, None) == -5
    assert gg(p, p, p, p, p, 4, B.GROUP_M, 512, 96, 128, 0, 0, 0, p, 1, None) == -5
    assert gg(p, p, p, p, p, 4, B.GROUP_K, 128, 128, 512, 0, 0, 0, p, 1, None) == -5    # GROUP_K needs token-major B
    assert gg(p, p, p, p, ctypes.c_void_p(0x1002), 4, B.GROUP_M, 512, 128, 128, 0, 0, 0, p, 1, None) == -4   # offsets need 4-byte alignment
    # linear-layer step
    ln = L.mxfp8_linear
    assert ln(p, p, p, 128, 128, 128, 0, p, p, p, None, 0, None) == -1
    assert ln(p, p, p, 96, 128, 128, 0, p, p, p, p, 1 << 30, None) == -5
    assert ln(p, p, p, 128, 128, 128, 7, p, p, p, p, 1 << 30, None) == -2
    assert ln(p, p, p, 128, 128, 128, 0, p, p, p, ctypes.c_void_p(0x1100), 16, None) == -8
    assert B.status_string(-9).startswith("invalid values")


def test_per_device_and_tensor_map_caches(tmp_path):
    """The status-word / SM-count caches hand every device its own entry (device index given explicitly, no
    GPU needed), and the tensor-map cache hits only on identical encode arguments."""
    import subprocess
    here = os.path.dirname(os.path.abspath(__file__))
    root = os.path.dirname(here)
    exe = str(tmp_path / "host_caches_test")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-I" + os.path.join(root, "paper_2506_08027_b200", "csrc"),
                           "-I" + os.path.join(cuda, "include"), os.path.join(here, "cpp", "host_caches_test.cpp"),
                           "-L" + os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + os.path.join(cuda, "lib64"), "-o", exe])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "all checks passed" in out.stdout
