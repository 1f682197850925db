"""Parity of mxfp8_gemm with the FP64 oracle over decoded operands.

Exact-integer cases must match exactly (every partial sum is an integer below 2^24, so any
FP32 accumulation order gives the same result); everything else must meet the tolerance:
relative Frobenius error <= 1e-5 and |D - D64| <= 2^-16 * sum_k |a_k b_k| per element.
"""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import gpu_gemm, check_gemm_tolerance

pytestmark = pytest.mark.gpu

INTS = np.array([-4, -3, -2, -1, 0, 1, 2, 3, 4])


def int_operand(rng, mn, k):
    vals = rng.choice(INTS, (mn, k))
    enc = np.zeros(256, dtype=np.uint8)
    for v in INTS:
        enc[int(v) & 0xFF] = orc.fp8_encode(float(v))
    return vals, enc[vals.astype(np.int64) & 0xFF]


def stored(q_logical, s_logical, major):
    """logical [MN,K] data and [MN,K/32] scales -> storage for 'k' or 'mn' majorness."""
    if major == "k":
        return q_logical, s_logical
    return np.ascontiguousarray(q_logical.T), np.ascontiguousarray(s_logical.T)


@pytest.mark.parametrize("shape", [(128, 128, 128), (128, 256, 128), (256, 128, 256), (384, 512, 640), (128, 384, 1024)])
@pytest.mark.parametrize("majors", [("k", "k"), ("k", "mn"), ("mn", "k"), ("mn", "mn")])
def test_exact_integers(shape, majors):
    m, n, k = shape
    rng = np.random.default_rng(m + 3 * n + 7 * k)
    ai, aq = int_operand(rng, m, k)
    bi, bq = int_operand(rng, n, k)
    a_s = np.full((m, k // 32), 127, np.uint8)
    b_s = np.full((n, k // 32), 127, np.uint8)
    want = (ai @ bi.T).astype(np.float64)
    A, SA = stored(aq, a_s, majors[0])
    B_, SB = stored(bq, b_s, majors[1])
    d64, _ = orc.gemm_f64(A, SA, B_, SB, majors[0], majors[1])
    assert np.array_equal(d64, want)
    got = gpu_gemm(A, SA, B_, SB, majors[0], majors[1])
    assert np.array_equal(got.astype(np.float64), want), "max |diff| = %g" % np.abs(got - want).max()


@pytest.mark.parametrize("majors", [("k", "k"), ("mn", "mn")])
def test_identity_b_returns_decoded_a(majors):
    # B = identity (K = N): D equals the decoded A exactly
    m, n = 256, 256
    k = n
    x = synth.gradient_like((m, k), 12)
    if majors[0] == "k":
        aq, a_s = orc.quantize(x, orc.ROW)
        a_dec = orc.dequantize_f64(aq, a_s, orc.ROW)
    else:
        aq, a_s = orc.quantize(np.ascontiguousarray(x.T), orc.COL)
        a_dec = orc.dequantize_f64(aq, a_s, orc.COL).T
    eye_q = np.where(np.eye(n, dtype=bool), orc.fp8_encode(1.0), 0).astype(np.uint8)
    eye_s = np.full((n, k // 32), 127, np.uint8)
    Bq, Bs = stored(eye_q, eye_s, majors[1])
    got = gpu_gemm(aq, a_s, Bq, Bs, majors[0], majors[1])
    assert np.array_equal(got.astype(np.float64), a_dec.astype(np.float32).astype(np.float64))


@pytest.mark.parametrize("majors", [("k", "k"), ("mn", "mn")])
def test_one_hot_scales_pin_the_scale_layout(majors):
    # all scale bytes 127 except one (mn, kb) = 128: exactly the products through that block
    # double.  Sweeps rows across quadrants / tiles and K-blocks across atoms and stages.
    m, n, k = 256, 256, 512
    rng = np.random.default_rng(4)
    ai, aq = int_operand(rng, m, k)
    bi, bq = int_operand(rng, n, k)
    base = (ai @ bi.T).astype(np.float64)
    picks = [(0, 0), (1, 1), (31, 3), (32, 4), (77, 5), (127, 15), (128, 0), (200, 9), (255, 15), (96, 7)]
    for which in ("a", "b"):
        for (mn, kb) in picks:
            a_s = np.full((m, k // 32), 127, np.uint8)
            b_s = np.full((n, k // 32), 127, np.uint8)
            extra = np.zeros((m, n))
            if which == "a":
                a_s[mn, kb] = 128
                extra[mn, :] = ai[mn, kb * 32:(kb + 1) * 32] @ bi[:, kb * 32:(kb + 1) * 32].T
            else:
                b_s[mn, kb] = 129
                extra[:, mn] = 3 * (ai[:, kb * 32:(kb + 1) * 32] @ bi[mn, kb * 32:(kb + 1) * 32])
            A, SA = stored(aq, a_s, majors[0])
            B_, SB = stored(bq, b_s, majors[1])
            got = gpu_gemm(A, SA, B_, SB, majors[0], majors[1])
            assert np.array_equal(got.astype(np.float64), base + extra), (which, mn, kb)


def test_pr1_reference_gemm():
    # config 1: both operands 256x512 FP32, quantized rowwise (paper rule), M=N=256, K=512;
    # and the same product from column-quantized transposes (MN-major x MN-major).
    a = synth.pr1_tensor(0)
    b = synth.pr1_tensor(1)
    aq, a_s = orc.quantize(a, orc.ROW)
    bq, b_s = orc.quantize(b, orc.ROW)
    d64, sabs = orc.gemm_f64(aq, a_s, bq, b_s)
    got = gpu_gemm(aq, a_s, bq, b_s)
    check_gemm_tolerance(got, d64, sabs, "pr1 k-major")
    aqt, a_st = orc.quantize(np.ascontiguousarray(a.T), orc.COL)
    bqt, b_st = orc.quantize(np.ascontiguousarray(b.T), orc.COL)
    assert np.array_equal(aqt.T, aq) and np.array_equal(a_st.T, a_s)
    got2 = gpu_gemm(aqt, a_st, bqt, b_st, "mn", "mn")
    check_gemm_tolerance(got2, d64, sabs, "pr1 mn-major")


@pytest.mark.parametrize("shape,majors", [((512, 768, 1024), ("k", "k")), ((256, 1280, 2048), ("k", "mn")),
                                          ((640, 256, 4096), ("mn", "mn")), ((1024, 1024, 512), ("mn", "k"))])
@pytest.mark.parametrize("elems", [(0, 0), (1, 0), (0, 1)])
def test_random_operands_meet_tolerance(shape, majors, elems):
    m, n, k = shape
    a = synth.gaussian((m, k), 100 + m)
    b = synth.output_gradient((n, k), 200 + n)
    qa = orc.quantize(a, orc.ROW, orc.RULE_PAPER, elems[0])
    qb = orc.quantize(b, orc.ROW, orc.RULE_PAPER, elems[1])
    A, SA = stored(qa[0], qa[1], majors[0])
    B_, SB = stored(qb[0], qb[1], majors[1])
    d64, sabs = orc.gemm_f64(A, SA, B_, SB, majors[0], majors[1], elems[0], elems[1])
    got = gpu_gemm(A, SA, B_, SB, majors[0], majors[1], elems[0], elems[1])
    check_gemm_tolerance(got, d64, sabs, str((shape, majors, elems)))


def test_bf16_output_is_rne_of_fp32_output_and_deterministic():
    import torch
    m, n, k = 384, 512, 1024
    a = synth.gaussian((m, k), 1)
    b = synth.gaussian((n, k), 2, 0.02)
    aq, a_s = orc.quantize(a, orc.ROW)
    bq, b_s = orc.quantize(b, orc.ROW)
    d32 = gpu_gemm(aq, a_s, bq, b_s)
    d32b = gpu_gemm(aq, a_s, bq, b_s)
    assert np.array_equal(d32.view(np.uint32), d32b.view(np.uint32))
    dbf = gpu_gemm(aq, a_s, bq, b_s, out="bf16")
    want = torch.from_numpy(d32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(dbf, want)
    d64, sabs = orc.gemm_f64(aq, a_s, bq, b_s)
    check_gemm_tolerance(d32, d64, sabs)


def test_nan_scale_byte_poisons_its_outputs():
    m, n, k = 128, 128, 256
    rng = np.random.default_rng(9)
    _, aq = int_operand(rng, m, k)
    _, bq = int_operand(rng, n, k)
    a_s = np.full((m, k // 32), 127, np.uint8)
    b_s = np.full((n, k // 32), 127, np.uint8)
    b_s[5, 2] = 0xFF
    d64, _ = orc.gemm_f64(aq, a_s, bq, b_s)
    got = gpu_gemm(aq, a_s, bq, b_s)
    assert np.array_equal(np.isnan(got), np.isnan(d64))


# ------------------------------------------------------------------------------- fused MXFP8 output

def _run_fused(aq, a_s, bq, b_s, orientation, rule, elem, with_d):
    """GEMM with the fused MXFP8 epilogue; returns dict of numpy outputs (raw swizzled scales)."""
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import swizzle_np
    M, K = aq.shape
    N = bq.shape[0]
    dA, dB = torch.from_numpy(aq).cuda(), torch.from_numpy(bq).cuda()
    dSA, dSB = torch.from_numpy(swizzle_np(a_s)).cuda(), torch.from_numpy(swizzle_np(b_s)).cuda()
    outs = {}
    bufs = []
    for o in (B.ROW, B.COL):
        if orientation & o:
            bufs.append(torch.zeros((M, N), dtype=torch.uint8, device="cuda"))
            bufs.append(torch.zeros(B.mxfp8_scale_bytes(M, N, o, B.SF_SWIZZLED), dtype=torch.uint8, device="cuda"))
        else:
            bufs += [None, None]
    epi = B.make_epilogue(orientation, rule, elem, *bufs)
    D = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") if with_d else None
    B.mxfp8_gemm(dA, dSA, dB, dSB, M, N, K, B.K_MAJOR, B.K_MAJOR, 0, 0, D, epi=epi)
    assert B.mxfp8_device_status() == 0
    names = ("q_row", "s_row", "q_col", "s_col")
    for n, b in zip(names, bufs):
        if b is not None:
            outs[n] = b.cpu().numpy()
    if D is not None:
        outs["D"] = D.cpu().numpy()
    return outs


@pytest.mark.parametrize("orientation", [1, 2, 3])
@pytest.mark.parametrize("rule", [orc.RULE_PAPER, orc.RULE_OCP])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_fused_epilogue_equals_quantize_of_unfused_output(orientation, rule, elem):
    # Sec. 2: the FP32 output is quantized to MX format when its consumer needs it.  The fused bytes must
    # be exactly what mxfp8_quantize (oracle-exact) makes of the same kernel's unfused FP32 output.
    import torch
    from paper_2506_08027_b200 import binding as B
    m, n, k = 512, 768, 512
    a = synth.gaussian((m, k), 7)
    b = synth.output_gradient((n, k), 8)
    aq, a_s = orc.quantize(a, orc.ROW)
    bq, b_s = orc.quantize(b, orc.ROW)
    d32 = gpu_gemm(aq, a_s, bq, b_s)                                   # unfused FP32 output
    fused = _run_fused(aq, a_s, bq, b_s, orientation, rule, elem, with_d=True)
    assert np.array_equal(fused["D"].view(np.uint32), d32.view(np.uint32))
    src = torch.from_numpy(d32).cuda()
    ref = B.alloc_quantize_outputs(m, n, orientation, B.SF_SWIZZLED)
    for t in ref:
        if t is not None:
            t.zero_()
    B.mxfp8_quantize(src, orientation, rule, elem, *ref, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    for name, t in zip(("q_row", "s_row", "q_col", "s_col"), ref):
        if t is not None:
            assert np.array_equal(fused[name], t.cpu().numpy()), name
    only = _run_fused(aq, a_s, bq, b_s, orientation, rule, elem, with_d=False)   # D = NULL
    for name in ("q_row", "s_row", "q_col", "s_col"):
        if name in fused:
            assert np.array_equal(only[name], fused[name]), name


def test_fused_epilogue_against_fp64_oracle():
    # decoded fused output vs the FP64 product: GEMM bound + one FP8 rounding (half an ulp of the element
    # grid relative, 2^-4 for E4M3, plus half the smallest subnormal times the block scale)
    from helpers import logical_scales_from_swizzled
    m, n, k = 256, 512, 1024
    a = synth.gaussian((m, k), 17)
    b = synth.gaussian((n, k), 18, 0.02)
    aq, a_s = orc.quantize(a, orc.ROW)
    bq, b_s = orc.quantize(b, orc.ROW)
    d64, sabs = orc.gemm_f64(aq, a_s, bq, b_s)
    fused = _run_fused(aq, a_s, bq, b_s, 3, orc.RULE_PAPER, orc.E4M3, with_d=False)
    s_row = logical_scales_from_swizzled(fused["s_row"], m, n // 32)             # [m, n/32]
    s_col = logical_scales_from_swizzled(fused["s_col"], n, m // 32).T           # [m/32, n]
    for q, s, orient in ((fused["q_row"], s_row, orc.ROW), (fused["q_col"], np.ascontiguousarray(s_col), orc.COL)):
        dq = orc.dequantize_f64(q, s, orient)
        x = np.exp2(s.astype(np.float64) - 127)
        xfull = np.repeat(x, 32, axis=1) if orient == orc.ROW else np.repeat(x, 32, axis=0)
        bound = 2.0 ** -16 * sabs + 2.0 ** -4 * np.abs(d64) * 1.001 + 2.0 ** -10 * xfull
        assert (np.abs(dq - d64) <= bound).all()
        # paper rule: nothing saturates (no decoded magnitude above 448 * X) and the scale is tight
        assert (np.abs(dq) <= 448 * xfull).all()


@pytest.mark.parametrize("shape", [(256, 384, 256), (384, 128, 128), (640, 896, 384)])
@pytest.mark.parametrize("tile", ["256p", "256", "128"])
def test_fused_epilogue_on_outputs_that_end_inside_a_tile(shape, tile, monkeypatch):
    """M and N are multiples of 128 but not of the tile: the warps whose columns or rows lie beyond the output must
    write nothing -- no element byte, no scale byte (guard bands around every buffer, pads zero)."""
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import Guarded, swizzle_np
    m, n, k = shape
    if tile == "256p" and m < 256:
        pytest.skip("a CTA pair needs 256 rows")
    monkeypatch.setenv("MXFP8_GEMM_TILE", tile)
    a = synth.gaussian((m, k), 21)
    b = synth.student_t((n, k), 22)
    aq, a_s = orc.quantize(a, orc.ROW)
    bq, b_s = orc.quantize(b, orc.ROW)
    dA, dB = torch.from_numpy(aq).cuda(), torch.from_numpy(bq).cuda()
    dSA, dSB = torch.from_numpy(swizzle_np(a_s)).cuda(), torch.from_numpy(swizzle_np(b_s)).cuda()
    g = [Guarded(m * n), Guarded(B.mxfp8_scale_bytes(m, n, B.ROW, B.SF_SWIZZLED)),
         Guarded(m * n), Guarded(B.mxfp8_scale_bytes(m, n, B.COL, B.SF_SWIZZLED))]
    for x in g:
        x.view.zero_()
    epi = B.make_epilogue(B.BOTH, B.RULE_PAPER, B.E4M3, g[0].view.view(m, n), g[1].view, g[2].view.view(m, n), g[3].view)
    D = torch.empty((m, n), dtype=torch.float32, device="cuda")
    B.mxfp8_gemm(dA, dSA, dB, dSB, m, n, k, B.K_MAJOR, B.K_MAJOR, 0, 0, D, epi=epi)
    assert B.mxfp8_device_status() == 0
    ref = B.alloc_quantize_outputs(m, n, B.BOTH, B.SF_SWIZZLED)
    for t in ref:
        t.zero_()
    B.mxfp8_quantize(D, B.BOTH, B.RULE_PAPER, B.E4M3, *ref, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    for name, got, want in zip(("q_row", "s_row", "q_col", "s_col"), g, ref):
        got.check(name)
        assert np.array_equal(got.numpy(), want.cpu().numpy().reshape(-1)), name


# ------------------------------------------------------------------------------- benchmark sizes

def test_bench_step_shapes_sampled_rows():
    """The three GEMMs of the benchmark step at full size (tokens 8192, hidden 2048, FFN 8192), in the
    launch configuration bench.py times.  Operands are quantized by the oracle on the host; 48 sampled
    output rows of each product (first, last, tile edges, random) are checked element by element against
    the FP64 oracle; the BF16 output must be the RNE rounding of the FP32 output."""
    import os
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import swizzle_np
    T, H, F = 8192, 2048, 8192
    thr = os.cpu_count() or 1
    x = synth.bf16_bits_as_f32(synth.f32_to_bf16_bits(synth.gaussian((T, H), synth.seed_for(2, 0))))
    w = synth.bf16_bits_as_f32(synth.f32_to_bf16_bits(synth.gaussian((F, H), synth.seed_for(2, 1), 0.02)))
    dy = synth.bf16_bits_as_f32(synth.f32_to_bf16_bits(synth.output_gradient((T, F), synth.seed_for(2, 2))))
    q = {}
    for name, t in (("x", x), ("w", w), ("dy", dy)):
        q[name, "r"] = orc.quantize_threads(t, orc.ROW, orc.RULE_PAPER, orc.E4M3, thr)
        q[name, "c"] = orc.quantize_threads(t, orc.COL, orc.RULE_PAPER, orc.E4M3, thr)
    dev = {}
    for key, (qq, ss) in q.items():
        s_log = ss if key[1] == "r" else np.ascontiguousarray(ss.T)
        dev[key] = (torch.from_numpy(qq).cuda(), torch.from_numpy(swizzle_np(s_log)).cuda())
    rng = np.random.default_rng(5)
    cases = (("fprop", ("x", "r"), ("w", "r"), "k", "k", T, F, H),
             ("dgrad", ("dy", "r"), ("w", "c"), "k", "mn", T, H, F),
             ("wgrad", ("dy", "c"), ("x", "c"), "mn", "mn", F, H, T))
    for name, ka, kb, am, bm, M, N, K in cases:
        rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, M - 257, M - 256, M - 129, M - 128, M - 1],
                                         rng.integers(0, M, 37)]))
        d32 = torch.empty((M, N), dtype=torch.float32, device="cuda")
        dbf = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        args = (dev[ka][0], dev[ka][1], dev[kb][0], dev[kb][1], M, N, K,
                B.MN_MAJOR if am == "mn" else B.K_MAJOR, B.MN_MAJOR if bm == "mn" else B.K_MAJOR, 0, 0)
        B.mxfp8_gemm(*args, d32)
        B.mxfp8_gemm(*args, dbf)
        assert B.mxfp8_device_status() == 0
        assert torch.equal(d32.to(torch.bfloat16), dbf), name
        aq, a_s = q[ka]
        if am == "k":
            a_sub, as_sub = aq[rows], a_s[rows]
        else:
            a_sub, as_sub = np.ascontiguousarray(aq[:, rows]), np.ascontiguousarray(a_s[:, rows])
        d64, sabs = orc.gemm_f64(a_sub, as_sub, q[kb][0], q[kb][1], am, bm)
        got = d32[torch.from_numpy(rows).cuda()].cpu().numpy()
        check_gemm_tolerance(got, d64, sabs, name)


@pytest.mark.parametrize("shape", [(200, 136, 160), (72, 264, 96), (1, 8, 32), (257, 520, 416), (384, 200, 2080), (130, 256, 128)])
@pytest.mark.parametrize("majors", [("k", "k"), ("k", "mn"), ("mn", "mn")])
def test_ragged_shapes(shape, majors):
    # M, N, K that are not multiples of the tile: out-of-range rows / columns / K are zero-filled on load
    # and clipped on store; the scale buffers are padded to whole atoms (pad bytes 0) as mxfp8_quantize writes them
    m, n, k = shape
    if majors[0] == "mn" and m % 16:
        pytest.skip("MN-major A needs M % 16 == 0")
    if majors[1] == "mn" and n % 16:
        pytest.skip("MN-major B needs N % 16 == 0")
    rng = np.random.default_rng(m * 7 + n * 3 + k)
    ai, aq = int_operand(rng, m, k)
    bi, bq = int_operand(rng, n, k)
    # unit scales: integer products, exact in FP32 for any accumulation order
    a_s = np.full((m, k // 32), 127, np.uint8)
    b_s = np.full((n, k // 32), 127, np.uint8)
    A, SA = stored(aq, a_s, majors[0])
    B_, SB = stored(bq, b_s, majors[1])
    got = gpu_gemm(A, SA, B_, SB, majors[0], majors[1])
    want = (ai @ bi.T).astype(np.float64)
    assert np.array_equal(got.astype(np.float64), want), "max |diff| = %g" % np.abs(got - want).max()
    # random scales: tolerance against the FP64 oracle
    a_s = rng.integers(110, 140, (m, k // 32)).astype(np.uint8)
    b_s = rng.integers(110, 140, (n, k // 32)).astype(np.uint8)
    A, SA = stored(aq, a_s, majors[0])
    B_, SB = stored(bq, b_s, majors[1])
    d64, sabs = orc.gemm_f64(A, SA, B_, SB, majors[0], majors[1])
    got = gpu_gemm(A, SA, B_, SB, majors[0], majors[1])
    check_gemm_tolerance(got, d64, sabs, str(shape))
    if n % 8 == 0:
        gotb = gpu_gemm(A, SA, B_, SB, majors[0], majors[1], out="bf16")
        import torch
        assert np.array_equal(gotb, torch.from_numpy(got).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def _multi_case(M, N, K, a_mn, b_mn, a_elem, b_elem, seed):
    """Operands quantized by the oracle; returns device tensors, problem tuple pieces and the FP64 result."""
    import torch
    from helpers import swizzle_np
    a = synth.gaussian((M, K), seed)
    b = synth.student_t((N, K), seed + 1) * np.float32(0.05)
    def prep(x, elem, mn):
        stored = np.ascontiguousarray(x.T) if mn else x
        q, s = orc.quantize(stored, orc.COL if mn else orc.ROW, orc.RULE_PAPER, elem)
        logical = np.ascontiguousarray(s.T) if mn else s
        return q, s, torch.from_numpy(orc.pack_codes16(q, elem)).cuda(), torch.from_numpy(swizzle_np(logical)).cuda()
    aq, a_s, da, dsa = prep(a, a_elem, a_mn)
    bq, b_s, db, dsb = prep(b, b_elem, b_mn)
    d64, sabs = orc.gemm_f64(aq, a_s, bq, b_s, "mn" if a_mn else "k", "mn" if b_mn else "k", a_elem, b_elem)
    return da, dsa, db, dsb, d64, sabs


@pytest.mark.parametrize("out", ["fp32", "bf16"])
def test_gemm_multi_equals_separate_products_and_oracle(out):
    # three products of different shapes, majors and element types (one ragged, one with 6-bit operands) in one
    # launch: each output equals the single-product launch bit for bit and the oracle within the tolerance
    import torch
    from paper_2506_08027_b200 import binding as B
    specs = [(512, 768, 256, False, False, orc.E4M3, orc.E4M3),
             (384, 256, 1024, False, True, orc.E5M2, orc.E4M3),
             (336, 208, 512, True, True, orc.E2M3, orc.E4M3)]
    dt = torch.float32 if out == "fp32" else torch.bfloat16
    cases, entries, outs = [], [], []
    for i, (M, N, K, a_mn, b_mn, ae, be) in enumerate(specs):
        c = _multi_case(M, N, K, a_mn, b_mn, ae, be, 40 + 3 * i)
        D = torch.full((M, N), float("nan"), dtype=dt, device="cuda")
        cases.append(c); outs.append(D)
        entries.append((c[0], c[1], c[2], c[3], M, N, K, int(a_mn), int(b_mn), ae, be, D))
    before = B.mxfp8_launch_count()
    B.mxfp8_gemm_multi(B.make_gemm_problems(entries), B.FP32 if out == "fp32" else B.BF16)
    assert B.mxfp8_device_status() == 0
    assert B.mxfp8_launch_count() - before == 1
    for (M, N, K, a_mn, b_mn, ae, be), c, D in zip(specs, cases, outs):
        single = torch.full((M, N), float("nan"), dtype=dt, device="cuda")
        B.mxfp8_gemm(c[0], c[1], c[2], c[3], M, N, K, int(a_mn), int(b_mn), ae, be, single)
        torch.cuda.synchronize()
        assert torch.equal(D.view(torch.int32 if out == "fp32" else torch.int16), single.view(torch.int32 if out == "fp32" else torch.int16))
        if out == "fp32":
            check_gemm_tolerance(D.cpu().numpy(), c[4], c[5], "multi %s" % ((M, N, K),))


def test_gemm_multi_many_tiles_and_uneven_depths():
    # the benchmark's mix in small: a shallow wide product and two deep narrow ones, more tiles than workers
    import torch
    from paper_2506_08027_b200 import binding as B
    specs = [(2048, 2048, 256, False, False), (2048, 512, 1024, False, True), (2048, 512, 1024, True, True)]
    entries, keep = [], []
    for i, (M, N, K, a_mn, b_mn) in enumerate(specs):
        c = _multi_case(M, N, K, a_mn, b_mn, orc.E4M3, orc.E4M3, 70 + 3 * i)
        D = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        keep.append((c, D))
        entries.append((c[0], c[1], c[2], c[3], M, N, K, int(a_mn), int(b_mn), orc.E4M3, orc.E4M3, D))
    B.mxfp8_gemm_multi(B.make_gemm_problems(entries), B.FP32)
    assert B.mxfp8_device_status() == 0
    for (M, N, K, _, _), (c, D) in zip(specs, keep):
        check_gemm_tolerance(D.cpu().numpy(), c[4], c[5], "multi deep %s" % ((M, N, K),))


def test_gemm_multi_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    z = torch.zeros(128, 128, dtype=torch.uint8, device="cuda")
    sc = torch.zeros(512, dtype=torch.uint8, device="cuda")
    D = torch.empty(128, 128, dtype=torch.float32, device="cuda")
    good = (z, sc, z, sc, 128, 128, 128, 0, 0, 0, 0, D)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_gemm_multi(B.make_gemm_problems([good] * 4), B.FP32)                 # more than three products
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_gemm_multi(B.make_gemm_problems([good, (z, sc, z, sc, 128, 128, 100, 0, 0, 0, 0, D)]), B.FP32)   # K % 32
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_gemm_multi(B.make_gemm_problems([good]), 7)                           # unknown output dtype


def test_output_with_more_than_2_to_31_elements_sampled():
    # D is 65536 x 40960 = 2.7e9 BF16 elements (5.4 GB); K is small so the oracle can check whole 128-row slabs
    import torch
    from paper_2506_08027_b200 import binding as B
    M, N, K = 65536, 40960, 256
    a = synth.device_tensor("activation", (M, K), 5)
    b = synth.device_tensor("weight", (N, K), 6)
    qa = B.alloc_quantize_outputs(M, K, B.ROW, B.SF_SWIZZLED)
    qb = B.alloc_quantize_outputs(N, K, B.ROW, B.SF_SWIZZLED)
    B.mxfp8_quantize(a, B.ROW, B.RULE_PAPER, B.E4M3, *qa, B.SF_SWIZZLED)
    B.mxfp8_quantize(b, B.ROW, B.RULE_PAPER, B.E4M3, *qb, B.SF_SWIZZLED)
    D = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    B.mxfp8_gemm(qa[0], qa[1], qb[0], qb[1], M, N, K, B.K_MAJOR, B.K_MAJOR, B.E4M3, B.E4M3, D)
    assert B.mxfp8_device_status() == 0
    bf = orc.bf16_bits_to_f32(b.view(torch.int16).cpu().numpy().view(np.uint16))
    bq, bs = orc.quantize(bf, orc.ROW)
    mark = (2 ** 31) // N // 128 * 128
    for r0 in (0, mark, M - 128):
        af = orc.bf16_bits_to_f32(a[r0:r0 + 128].view(torch.int16).cpu().numpy().view(np.uint16))
        aq, a_s = orc.quantize(af, orc.ROW)
        d64, sabs = orc.gemm_f64(aq, a_s, bq, bs)
        got = orc.bf16_bits_to_f32(D[r0:r0 + 128].view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
        err = np.abs(got - d64)
        assert (err <= 2.0 ** -16 * sabs + 2.0 ** -8 * np.abs(d64) + 2.0 ** -126).all(), "slab %d" % r0


@pytest.mark.parametrize("majors", [("k", "k"), ("mn", "mn")])
def test_k_permutation_leaves_exact_products_unchanged(majors):
    # the same permutation of the K axis in both operands (elements together with their blocks' scales): shuffling
    # inside blocks, shuffling whole blocks, and both.  Small integers and power-of-two scales keep every partial
    # sum exact in FP32, so the result must not change by a single bit, whatever the order of accumulation.
    m, n, k = 256, 384, 512
    rng = np.random.default_rng(91)
    ai, aq = int_operand(rng, m, k)
    bi, bq = int_operand(rng, n, k)
    a_s = rng.integers(126, 129, (m, k // 32)).astype(np.uint8)      # 1/2, 1, 2: sums stay below 2^24 units
    b_s = rng.integers(126, 129, (n, k // 32)).astype(np.uint8)
    base = gpu_gemm(*stored(aq, a_s, majors[0]), *stored(bq, b_s, majors[1]), majors[0], majors[1])
    d64, _ = orc.gemm_f64(*stored(aq, a_s, majors[0]), *stored(bq, b_s, majors[1]), majors[0], majors[1])
    assert np.array_equal(base.astype(np.float64), d64)
    within = np.concatenate([32 * b + rng.permutation(32) for b in range(k // 32)])     # inside each block
    blocks = rng.permutation(k // 32)
    across = np.concatenate([32 * b + np.arange(32) for b in blocks])                   # whole blocks
    for perm, sperm in ((within, np.arange(k // 32)), (across, blocks), (across[within], blocks)):
        if perm is not within and perm is not across:
            # across[within]: first shuffle inside blocks, then move the blocks
            perm = np.concatenate([32 * b + rng.permutation(32) for b in blocks])
        got = gpu_gemm(*stored(aq[:, perm], a_s[:, sperm], majors[0]), *stored(bq[:, perm], b_s[:, sperm], majors[1]),
                       majors[0], majors[1])
        assert np.array_equal(got, base)


def test_bench_step_joint_launch_equals_single_launches_at_full_size():
    # the benchmark's GEMM launch: fprop + dgrad + wgrad (tokens 8192, hidden 2048, FFN 8192) as one pool of tiles.
    # Every output must equal, bit for bit, the single-product launch that test_bench_step_shapes_sampled_rows
    # checks against the oracle.
    import torch
    from paper_2506_08027_b200 import binding as B
    T, H, F = 8192, 2048, 8192
    E, S = B.E4M3, B.SF_SWIZZLED
    X = synth.device_tensor("activation", (T, H), synth.seed_for(2, 0))
    W = synth.device_tensor("weight", (F, H), synth.seed_for(2, 1))
    dY = synth.device_tensor("output_gradient", (T, F), synth.seed_for(2, 2))
    qX, qW, qdY = (B.alloc_quantize_outputs(t.shape[0], t.shape[1], B.BOTH, S) for t in (X, W, dY))
    B.mxfp8_quantize_multi(B.make_quantize_items([(X,) + qX, (W,) + qW, (dY,) + qdY]), B.BF16, B.BOTH, B.RULE_PAPER, E, S)
    specs = [(qX[0], qX[1], qW[0], qW[1], T, F, H, B.K_MAJOR, B.K_MAJOR),
             (qdY[0], qdY[1], qW[2], qW[3], T, H, F, B.K_MAJOR, B.MN_MAJOR),
             (qdY[2], qdY[3], qX[2], qX[3], F, H, T, B.MN_MAJOR, B.MN_MAJOR)]
    joint = [torch.full((m, n), float("nan"), dtype=torch.bfloat16, device="cuda") for (_, _, _, _, m, n, _, _, _) in specs]
    B.mxfp8_gemm_multi(B.make_gemm_problems([s + (E, E, d) for s, d in zip(specs, joint)]), B.BF16)
    assert B.mxfp8_device_status() == 0
    for (aq, a_s, bq, b_s, m, n, k, am, bm), d in zip(specs, joint):
        single = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.mxfp8_gemm(aq, a_s, bq, b_s, m, n, k, am, bm, E, E, single)
        torch.cuda.synchronize()
        assert torch.equal(d.view(torch.int16), single.view(torch.int16))


@pytest.mark.parametrize("case", ["ffn_up fprop", "qkv wgrad"])
def test_fused_output_at_decoder_block_sizes_equals_quantize_of_unfused_output(case):
    # two GEMMs of the 8B-class decoder block at full size (tokens 16384): the fused row+column MXFP8 output must
    # be byte for byte what mxfp8_quantize makes of the same product's FP32 output (all on the device)
    import torch
    from paper_2506_08027_b200 import binding as B
    E, S = B.E4M3, B.SF_SWIZZLED
    Tk = 16384
    if case == "ffn_up fprop":
        M, N, K, am, bm = Tk, 28672, 4096, B.K_MAJOR, B.K_MAJOR
        a = synth.device_tensor("activation", (M, K), 41)
        b = synth.device_tensor("weight", (N, K), 42)
        qa = B.alloc_quantize_outputs(M, K, B.ROW, S); B.mxfp8_quantize(a, B.ROW, B.RULE_PAPER, E, *qa, S)
        qb = B.alloc_quantize_outputs(N, K, B.ROW, S); B.mxfp8_quantize(b, B.ROW, B.RULE_PAPER, E, *qb, S)
        ops = (qa[0], qa[1], qb[0], qb[1])
    else:
        M, N, K, am, bm = 6144, 4096, Tk, B.MN_MAJOR, B.MN_MAJOR            # dW = dY^T X, both operands token-major
        dy = synth.device_tensor("output_gradient", (K, M), 43)
        x = synth.device_tensor("activation", (K, N), 44)
        qa = B.alloc_quantize_outputs(K, M, B.COL, S); B.mxfp8_quantize(dy, B.COL, B.RULE_PAPER, E, *qa, S)
        qb = B.alloc_quantize_outputs(K, N, B.COL, S); B.mxfp8_quantize(x, B.COL, B.RULE_PAPER, E, *qb, S)
        ops = (qa[2], qa[3], qb[2], qb[3])
    d32 = torch.empty((M, N), dtype=torch.float32, device="cuda")
    B.mxfp8_gemm(*ops, M, N, K, am, bm, E, E, d32)
    ref = B.alloc_quantize_outputs(M, N, B.BOTH, S)
    B.mxfp8_quantize(d32, B.BOTH, B.RULE_PAPER, E, *ref, S)
    fused = B.alloc_quantize_outputs(M, N, B.BOTH, S)
    for t in fused:
        t.zero_()
    epi = B.make_epilogue(B.BOTH, B.RULE_PAPER, E, *fused)
    d16 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    B.mxfp8_gemm(*ops, M, N, K, am, bm, E, E, d16, epi=epi)
    assert B.mxfp8_device_status() == 0
    for name, u, v in zip(("q_row", "s_row", "q_col", "s_col"), fused, ref):
        assert torch.equal(u, v), name
    assert torch.equal(d16, d32.to(torch.bfloat16))


@pytest.mark.parametrize("tile", ["256p", "192p", "256", "192", "128"])
@pytest.mark.parametrize("majors", [("k", "k"), ("mn", "mn")])
def test_every_tile_shape_against_the_oracle(tile, majors):
    # the tile shape is normally chosen by a cost model; here each of the five kernel shapes is forced in turn on a
    # product with ragged M, N and K tails (several tiles in both directions, two K blocks plus a tail)
    import os
    m, n, k = 656, 720, 352
    a = synth.gaussian((m, k), 61)
    b = synth.student_t((n, k), 62) * np.float32(0.1)
    def prep(x, major):
        stored_x = np.ascontiguousarray(x.T) if major == "mn" else x
        return orc.quantize(stored_x, orc.COL if major == "mn" else orc.ROW)
    aq, a_s = prep(a, majors[0])
    bq, b_s = prep(b, majors[1])
    d64, sabs = orc.gemm_f64(aq, a_s, bq, b_s, majors[0], majors[1])
    old = os.environ.pop("MXFP8_GEMM_TILE", None)
    os.environ["MXFP8_GEMM_TILE"] = tile
    try:
        got = gpu_gemm(aq, a_s, bq, b_s, majors[0], majors[1])
    finally:
        os.environ.pop("MXFP8_GEMM_TILE", None)
        if old is not None:
            os.environ["MXFP8_GEMM_TILE"] = old
    check_gemm_tolerance(got, d64, sabs, "tile %s %s" % (tile, majors))


def test_clock_probe_reports_a_plausible_sm_clock():
    """The kernel's own cycles / wall time: between the idle floor and the boost clock, for a launch long enough to measure."""
    import torch
    from paper_2506_08027_b200 import binding as B
    n = 4096
    q = torch.zeros(n, n, dtype=torch.uint8, device="cuda")
    sf = torch.full((B.mxfp8_scale_bytes(n, n, B.ROW, B.SF_SWIZZLED),), 127, dtype=torch.uint8, device="cuda")
    d = torch.empty(n, n, dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        B.mxfp8_gemm(q, sf, q, sf, n, n, n, B.K_MAJOR, B.K_MAJOR, B.E4M3, B.E4M3, d)
    mhz, us = B.mxfp8_gemm_last_clock()
    assert 300.0 < mhz < 2500.0 and 5.0 < us < 5000.0, (mhz, us)
