"""mxfp8_grouped_gemm (per-expert products of a mixture-of-experts layer, App. A.4) against the oracle."""
import os

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import swizzle_np, check_gemm_tolerance

pytestmark = pytest.mark.gpu


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_grouped(aq, a_log, bq, b_log, offsets, mode, M, N, K, b_major, d_rows, out="fp32", tile=None):
    """a_log / b_log: logical [MN, K/32] scale matrices.  Returns (D numpy with NaN where nothing was stored, status)."""
    import torch
    from paper_2506_08027_b200 import binding as B
    D = torch.full((d_rows, N), float("nan"), dtype=torch.float32 if out == "fp32" else torch.bfloat16, device="cuda")
    off = torch.tensor(offsets, dtype=torch.int32, device="cuda")
    old = os.environ.pop("MXFP8_GEMM_TILE", None)
    if tile:
        os.environ["MXFP8_GEMM_TILE"] = tile
    try:
        B.mxfp8_grouped_gemm(dev(aq), dev(swizzle_np(a_log)), dev(bq), dev(swizzle_np(b_log)), off,
                             B.GROUP_M if mode == "m" else B.GROUP_K, M, N, K,
                             B.MN_MAJOR if b_major == "mn" else B.K_MAJOR, B.E4M3, B.E4M3, D)
    finally:
        os.environ.pop("MXFP8_GEMM_TILE", None)
        if old is not None:
            os.environ["MXFP8_GEMM_TILE"] = old
    status = B.mxfp8_device_status()
    if out == "fp32":
        return D.cpu().numpy(), status
    return orc.bf16_bits_to_f32(D.view(torch.int16).cpu().numpy().view(np.uint16)), status


def fprop_case(T, K, N, offsets, seed, b_major):
    """Tokens X [T, K] and G stacked expert matrices, quantized by the oracle."""
    G = len(offsets) - 1
    x = synth.gaussian((T, K), seed)
    aq, a_s = orc.quantize(x, orc.ROW, orc.RULE_PAPER, orc.E4M3)
    if b_major == "k":
        w = 0.05 * synth.student_t((G * N, K), seed + 1)
        bq, b_s = orc.quantize(w, orc.ROW, orc.RULE_PAPER, orc.E4M3)
        b_log = b_s                                     # [G*N, K/32]
    else:
        w = 0.05 * synth.student_t((G * K, N), seed + 1)
        bq, b_s = orc.quantize(w, orc.COL, orc.RULE_PAPER, orc.E4M3)
        b_log = np.ascontiguousarray(b_s.T)             # [N, G*K/32]
    return aq, a_s, bq, b_s, b_log


def check_rows(d, d64, sabs, offsets, what):
    lo, hi = offsets[0], offsets[-1]
    assert np.isnan(d[:lo]).all() and np.isnan(d[hi:]).all(), "rows outside every group were written " + what
    if hi > lo:
        check_gemm_tolerance(d[lo:hi], d64[lo:hi], sabs[lo:hi], what)


OFFSETS = {
    "even": [0, 256, 512, 768, 1024],
    "ragged": [0, 128, 128, 512, 896],            # an empty expert, odd 128-blocks, tokens 896.. unowned
    "late_start": [128, 384, 384, 1024],          # tokens 0..127 unowned
    "one": [0, 1024],
}


@pytest.mark.parametrize("name", list(OFFSETS))
@pytest.mark.parametrize("b_major", ["k", "mn"])
@pytest.mark.parametrize("tile", ["256p", "256"])
def test_group_m_against_oracle(name, b_major, tile):
    offsets = OFFSETS[name]
    T, K, N = 1024, 256, 384
    aq, a_s, bq, b_s, b_log = fprop_case(T, K, N, offsets, 50 + len(name), b_major)
    d, status = run_grouped(aq, a_s, bq, b_log, offsets, "m", T, N, K, b_major, T, tile=tile)
    assert status == 0
    d64, sabs = orc.grouped_gemm_f64(aq, a_s, bq, b_s, offsets, "m", b_major)
    check_rows(d, d64, sabs, offsets, "%s %s %s" % (name, b_major, tile))


@pytest.mark.parametrize("name", ["even", "ragged", "late_start"])
@pytest.mark.parametrize("tile", ["256p", "256"])
def test_group_k_against_oracle(name, tile):
    offsets = OFFSETS[name]
    G = len(offsets) - 1
    T, M, N = 1024, 384, 256
    dy = synth.output_gradient((T, M), 7)
    x = synth.gaussian((T, N), 8)
    aq, a_s = orc.quantize(dy, orc.COL, orc.RULE_PAPER, orc.E4M3)      # scales [T/32, M]
    bq, b_s = orc.quantize(x, orc.COL, orc.RULE_PAPER, orc.E4M3)
    d, status = run_grouped(aq, np.ascontiguousarray(a_s.T), bq, np.ascontiguousarray(b_s.T), offsets, "k",
                            M, N, T, "mn", G * M, tile=tile)
    assert status == 0
    d64, sabs = orc.grouped_gemm_f64(aq, a_s, bq, b_s, offsets, "k")
    check_gemm_tolerance(d, d64, sabs, "%s %s" % (name, tile))
    for g in range(G):
        if offsets[g] == offsets[g + 1]:
            assert not d[g * M:(g + 1) * M].any(), "an expert without tokens must produce zeros"


def test_exact_small_integers_both_modes():
    # unit scales and small integer elements: every product is an integer FP32 holds exactly
    rng = np.random.default_rng(3)
    ints = np.array([-3, -2, -1, 0, 1, 2, 3])
    enc = np.zeros(7, np.uint8)
    for i, v in enumerate(ints):
        enc[i] = orc.fp8_encode(float(v))
    offsets = [0, 384, 512, 512, 1280]
    G, T, K, N = 4, 1280, 128, 256
    ai, bi = rng.integers(0, 7, (T, K)), rng.integers(0, 7, (G * N, K))
    aq, bq = enc[ai], enc[bi]
    one = lambda r, c: np.full((r, c), 127, np.uint8)
    d, status = run_grouped(aq, one(T, K // 32), bq, one(G * N, K // 32), offsets, "m", T, N, K, "k", T)
    assert status == 0
    av, bv = ints[ai].astype(np.int64), ints[bi].astype(np.int64)
    for g in range(G):
        lo, hi = offsets[g], offsets[g + 1]
        assert np.array_equal(d[lo:hi], (av[lo:hi] @ bv[g * N:(g + 1) * N].T).astype(np.float32))
    # wgrad: D_g = A_g^T B_g with A [T, M], B [T, N]
    M = 128
    xi, yi = rng.integers(0, 7, (T, M)), rng.integers(0, 7, (T, N))
    d, status = run_grouped(enc[xi], one(M, T // 32), enc[yi], one(N, T // 32), offsets, "k", M, N, T, "mn", G * M)
    assert status == 0
    xv, yv = ints[xi].astype(np.int64), ints[yi].astype(np.int64)
    for g in range(G):
        lo, hi = offsets[g], offsets[g + 1]
        assert np.array_equal(d[g * M:(g + 1) * M], (xv[lo:hi].T @ yv[lo:hi]).astype(np.float32))


def test_bf16_output_is_rounded_fp32_output():
    offsets = OFFSETS["ragged"]
    T, K, N = 1024, 256, 384
    aq, a_s, bq, b_s, b_log = fprop_case(T, K, N, offsets, 99, "k")
    d32, _ = run_grouped(aq, a_s, bq, b_log, offsets, "m", T, N, K, "k", T)
    d16, status = run_grouped(aq, a_s, bq, b_log, offsets, "m", T, N, K, "k", T, out="bf16")
    assert status == 0
    inside = slice(offsets[0], offsets[-1])
    want = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(d32[inside]))
    assert np.array_equal(d16[inside], want)


def test_many_small_experts_and_many_tiles():
    # 64 experts of 128..640 tokens, several N tiles and K blocks: every worker walks many groups
    rng = np.random.default_rng(17)
    sizes = rng.integers(1, 6, 64) * 128
    sizes[5] = 0
    offsets = [0] + np.cumsum(sizes).tolist()
    T, K, N = int(offsets[-1]) + 128, 384, 640
    G = 64
    x = synth.gaussian((T, K), 1)
    aq, a_s = orc.quantize(x, orc.ROW, orc.RULE_PAPER, orc.E4M3)
    w = 0.05 * synth.gaussian((G * N, K), 2)
    bq, b_s = orc.quantize(w, orc.ROW, orc.RULE_PAPER, orc.E4M3)
    d64, sabs = orc.grouped_gemm_f64(aq, a_s, bq, b_s, offsets, "m", "k")
    for tile in ("256p", "256"):
        d, status = run_grouped(aq, a_s, bq, b_s, offsets, "m", T, N, K, "k", T, tile=tile)
        assert status == 0
        check_rows(d, d64, sabs, offsets, "64 experts " + tile)


@pytest.mark.parametrize("offsets", [[0, 100, 256], [0, 256, 128], [0, 128, 2048], [-128, 128, 256]])
def test_bad_offsets_are_reported_and_store_nothing(offsets):
    from paper_2506_08027_b200 import binding as B
    T, K, N = 1024, 128, 128
    G = len(offsets) - 1
    aq = np.zeros((T, K), np.uint8)
    bq = np.zeros((G * N, K), np.uint8)
    one = lambda r, c: np.full((r, c), 127, np.uint8)
    d, status = run_grouped(aq, one(T, K // 32), bq, one(G * N, K // 32), offsets, "m", T, N, K, "k", T)
    assert status == B.ERR_DEVICE_ARGS
    assert np.isnan(d).all()
    assert B.mxfp8_device_status() == 0          # reading the status clears it


def test_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    z = lambda *s: torch.zeros(*s, dtype=torch.uint8, device="cuda")
    off = torch.tensor([0, 128], dtype=torch.int32, device="cuda")
    D = torch.empty(128, 128, dtype=torch.float32, device="cuda")
    sc = z(512)
    with pytest.raises(B.Mxfp8Error):      # N not a multiple of 128
        B.mxfp8_grouped_gemm(z(128, 128), sc, z(64, 128), sc, off, B.GROUP_M, 128, 64, 128, B.K_MAJOR, B.E4M3, B.E4M3, D)
    with pytest.raises(B.Mxfp8Error):      # GROUP_K needs token-major B
        B.mxfp8_grouped_gemm(z(128, 128), sc, z(128, 128), sc, off, B.GROUP_K, 128, 128, 128, B.K_MAJOR, B.E4M3, B.E4M3, D)
    with pytest.raises(B.Mxfp8Error):      # unknown mode
        B.mxfp8_grouped_gemm(z(128, 128), sc, z(128, 128), sc, off, 3, 128, 128, 128, B.K_MAJOR, B.E4M3, B.E4M3, D)
    big = torch.zeros(300, dtype=torch.int32, device="cuda")
    with pytest.raises(B.Mxfp8Error):      # more than 256 experts
        B.mxfp8_grouped_gemm(z(128, 128), sc, z(128, 128), sc, big, B.GROUP_M, 128, 128, 128, B.K_MAJOR, B.E4M3, B.E4M3, D)


def test_no_tokens_at_all():
    # every expert empty: the token-grouped product stores nothing, the reduction-grouped one stores zeros
    T, K, N = 256, 128, 128
    offsets = [128, 128, 128, 128]
    G = 3
    one = lambda r, c: np.full((r, c), 127, np.uint8)
    aq = np.full((T, K), 0x38, np.uint8)
    bq = np.full((G * N, K), 0x38, np.uint8)
    d, status = run_grouped(aq, one(T, K // 32), bq, one(G * N, K // 32), offsets, "m", T, N, K, "k", T)
    assert status == 0 and np.isnan(d).all()
    M = 128
    d, status = run_grouped(np.full((T, M), 0x38, np.uint8), one(M, T // 32), np.full((T, N), 0x38, np.uint8), one(N, T // 32),
                            offsets, "k", M, N, T, "mn", G * M)
    assert status == 0 and not d.any() and not np.isnan(d).any()
