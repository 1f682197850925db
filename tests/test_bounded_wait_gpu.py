"""A bounded device wait that runs out, watched from the host.

Every mbarrier wait in the GEMM and conversion kernels has a time limit; when it passes, the kernel
records MXFP8_ERR_DEVICE_TIMEOUT in the device status word, all roles of the CTA leave, TMEM is
released and the context stays usable.  These tests run that path for real, in the one form that
cannot hang or fault anything: a test build of the library (-DMXFP8_TEST_HOOKS, its own .so, never
loaded by the binding) whose limit is 5 ms and whose producer can be told, through an environment
variable, to leave out the loads of one pipeline stage.  Nothing is in flight for that stage (the
copies were never issued), the consumer's wait runs out, the kernel returns.
"""
import ctypes
import os

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import swizzle_np

pytestmark = pytest.mark.gpu

TIMEOUT = -7


@pytest.fixture(scope="module")
def hooks():
    from paper_2506_08027_b200 import binding as B, build
    return B.load_library(build.build(test_hooks=True))


def _gemm(H, da, dsa, db, dsb, M, N, K, D):
    rc = H.mxfp8_gemm(da.data_ptr(), dsa.data_ptr(), db.data_ptr(), dsb.data_ptr(), M, N, K, 0, 0, 0, 0,
                      D.data_ptr(), 0, None, None, 0, None)
    assert rc == 0


def test_gemm_wait_runs_out_once_and_the_next_product_is_right(hooks, monkeypatch):
    import torch
    H = hooks
    M = N = 128
    K = 512                                   # four K blocks on one 128 x 128 tile of one CTA
    monkeypatch.setenv("MXFP8_GEMM_TILE", "128")
    rng = np.random.default_rng(3)
    ints = rng.integers(-4, 5, (M, K)), rng.integers(-4, 5, (N, K))
    enc = lambda v: np.vectorize(lambda x: orc.fp8_encode(float(x)), otypes=[np.uint8])(v)
    aq, bq = enc(ints[0]), enc(ints[1])
    ones = np.full((M, K // 32), 127, np.uint8)
    da, db = torch.from_numpy(aq).cuda(), torch.from_numpy(bq).cuda()
    dsa = torch.from_numpy(swizzle_np(ones)).cuda()
    dsb = torch.from_numpy(swizzle_np(ones)).cuda()
    D = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    assert H.mxfp8_device_status(None) == 0

    monkeypatch.setenv("MXFP8_TEST_SKIP_LOAD", "2")     # the loads of the second K block are never issued
    _gemm(H, da, dsa, db, dsb, M, N, K, D)
    assert H.mxfp8_device_status(None) == TIMEOUT       # reported once ...
    assert H.mxfp8_device_status(None) == 0             # ... and cleared by the read
    monkeypatch.delenv("MXFP8_TEST_SKIP_LOAD")

    # the context is intact: the same product, now complete, is exact (integer operands, unit scales)
    _gemm(H, da, dsa, db, dsb, M, N, K, D)
    assert H.mxfp8_device_status(None) == 0
    want = (ints[0] @ ints[1].T).astype(np.float64)
    assert np.array_equal(D.cpu().numpy().astype(np.float64), want)

    # a CTA pair gives up the same way (both CTAs leave, TMEM released by the pair)
    monkeypatch.setenv("MXFP8_GEMM_TILE", "256p")
    M2 = 256
    a2 = np.concatenate([aq, aq]); s2 = np.concatenate([ones, ones])
    da2, dsa2 = torch.from_numpy(a2).cuda(), torch.from_numpy(swizzle_np(s2)).cuda()
    D2 = torch.zeros((M2, N), dtype=torch.float32, device="cuda")
    monkeypatch.setenv("MXFP8_TEST_SKIP_LOAD", "3")
    _gemm(H, da2, dsa2, db, dsb, M2, N, K, D2)
    assert H.mxfp8_device_status(None) == TIMEOUT
    monkeypatch.delenv("MXFP8_TEST_SKIP_LOAD")
    _gemm(H, da2, dsa2, db, dsb, M2, N, K, D2)
    assert H.mxfp8_device_status(None) == 0
    assert np.array_equal(D2.cpu().numpy().astype(np.float64), np.concatenate([want, want]))


def test_conversion_wait_runs_out_once_and_the_next_conversion_is_right(hooks, monkeypatch):
    import torch
    from paper_2506_08027_b200 import binding as B
    H = hooks
    rows, cols = 256, 256                     # four tiles of 128 rows x 128 BF16 columns
    bits = synth.f32_to_bf16_bits(synth.gaussian((rows, cols), 17))
    src = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    q = torch.zeros((rows, cols), dtype=torch.uint8, device="cuda")
    s = torch.zeros(B.mxfp8_scale_bytes(rows, cols, B.ROW, B.SF_LINEAR), dtype=torch.uint8, device="cuda")

    def convert():
        rc = H.mxfp8_quantize(src.data_ptr(), B.BF16, rows, cols, B.ROW, B.RULE_PAPER, B.E4M3, q.data_ptr(), s.data_ptr(),
                              None, None, B.SF_LINEAR, None)
        assert rc == 0

    monkeypatch.setenv("MXFP8_TEST_SKIP_TILE", "2")     # the load of the second tile is never issued
    convert()
    assert H.mxfp8_device_status(None) == TIMEOUT
    assert H.mxfp8_device_status(None) == 0
    monkeypatch.delenv("MXFP8_TEST_SKIP_TILE")
    convert()
    assert H.mxfp8_device_status(None) == 0
    wq, ws = orc.quantize(orc.bf16_bits_to_f32(bits), orc.ROW)
    assert np.array_equal(q.cpu().numpy(), wq)
    assert np.array_equal(s.cpu().numpy().reshape(rows, cols // 32), ws)


def test_conversion_wait_runs_out_with_the_tile_counter_in_use(hooks, monkeypatch):
    """The same on a tensor large enough for tiles to be handed out through the stream's counter (more than four per
    CTA): the CTA whose load is left out gives up, the others finish, the last one out leaves the counter at zero,
    and the next conversion on the same stream is right."""
    import torch
    from paper_2506_08027_b200 import binding as B
    H = hooks
    rows, cols = 4096, 8192                   # 2048 tiles of 128 x 128
    bits = synth.f32_to_bf16_bits(synth.gaussian((rows, cols), 23))
    src = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    q = torch.zeros((rows, cols), dtype=torch.uint8, device="cuda")
    s = torch.zeros(B.mxfp8_scale_bytes(rows, cols, B.ROW, B.SF_LINEAR), dtype=torch.uint8, device="cuda")

    def convert():
        rc = H.mxfp8_quantize(src.data_ptr(), B.BF16, rows, cols, B.ROW, B.RULE_PAPER, B.E4M3, q.data_ptr(), s.data_ptr(),
                              None, None, B.SF_LINEAR, None)
        assert rc == 0

    convert()                                                   # a clean run first: the counter is back at zero after it
    assert H.mxfp8_device_status(None) == 0
    monkeypatch.setenv("MXFP8_TEST_SKIP_TILE", "700")           # whichever CTA is handed tile 699 never gets its data
    convert()
    assert H.mxfp8_device_status(None) == TIMEOUT
    assert H.mxfp8_device_status(None) == 0
    monkeypatch.delenv("MXFP8_TEST_SKIP_TILE")
    for _ in range(2):
        q.zero_(); s.zero_()
        convert()
        assert H.mxfp8_device_status(None) == 0
    wq, ws = orc.quantize_threads(orc.bf16_bits_to_f32(bits), orc.ROW, orc.RULE_PAPER, orc.E4M3, os.cpu_count() or 1)
    assert np.array_equal(q.cpu().numpy(), wq)
    assert np.array_equal(s.cpu().numpy().reshape(rows, cols // 32), ws)
