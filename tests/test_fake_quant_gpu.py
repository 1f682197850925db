"""Parity of mxfp8_fake_quantize (the MXFP8 round trip of Sec. 3.1) with the CPU oracle:
the output must equal dequantize(quantize(x)) of the oracle bit for bit, NaNs matching by position."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import Guarded

pytestmark = pytest.mark.gpu

ROW, COL, BOTH = 1, 2, 3


def gpu_fake_quantize(src_np, dtype, orientation, rule, elem):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = src_np.shape
    esz = 2 if dtype == "bf16" else 4
    if dtype == "bf16":
        src = torch.from_numpy(src_np.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        src = torch.from_numpy(src_np).cuda()
    bufs, args = {}, []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            bufs[name] = Guarded(rows * cols * esz)
            args.append(bufs[name].view)
        else:
            args.append(None)
    B.mxfp8_fake_quantize(src, orientation, rule, elem, args[0], args[1])
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    out = {}
    for name, g in bufs.items():
        g.check("dst_" + name)
        out[name] = g.numpy().view(np.uint16 if dtype == "bf16" else np.float32).reshape(rows, cols)
    return out


def oracle_round_trip(src_np, dtype, o, rule, elem):
    x = orc.bf16_bits_to_f32(src_np) if dtype == "bf16" else src_np
    q, s = orc.quantize(x, o, rule, elem)
    return orc.dequantize(q, s, o, elem, "bf16" if dtype == "bf16" else "f32")


def assert_same_values(got, want, dtype, what):
    if dtype == "bf16":
        g_nan = (got & 0x7FFF) > 0x7F80
        w_nan = (want & 0x7FFF) > 0x7F80
        g, w = got, want
    else:
        g_nan, w_nan = np.isnan(got), np.isnan(want)
        g, w = got.view(np.uint32), want.view(np.uint32)
    assert np.array_equal(g_nan, w_nan), "NaN positions differ " + what
    bad = (g != w) & ~g_nan
    assert not bad.any(), "%d values differ %s; first at %s" % (bad.sum(), what, np.argwhere(bad)[:4].tolist())


def check(src_np, dtype, orientation, rule, elem, what=""):
    got = gpu_fake_quantize(src_np, dtype, orientation, rule, elem)
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        if name in got:
            assert_same_values(got[name], oracle_round_trip(src_np, dtype, o, rule, elem), dtype, "(%s) %s" % (name, what))
    return got


def as_dtype(x32, dtype):
    return synth.f32_to_bf16_bits(x32) if dtype == "bf16" else x32


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("rule", [orc.RULE_PAPER, orc.RULE_OCP])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_pr1_reference_tensor(dtype, rule, elem):
    x = as_dtype(synth.pr1_tensor(0), dtype)
    for o in (ROW, COL, BOTH):
        check(x, dtype, o, rule, elem, "pr1 o=%d" % o)


@pytest.mark.parametrize("shape", [(32, 32), (1, 32), (7, 64), (160, 352), (128, 128), (160, 416), (384, 8288), (1024, 4096)])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_shapes_and_ragged_tiles(shape, dtype):
    rows, cols = shape
    x = as_dtype(synth.gaussian(shape, 4321 + rows + cols), dtype)
    for o in ([ROW] + ([COL, BOTH] if rows % 32 == 0 else [])):
        check(x, dtype, o, orc.RULE_PAPER, orc.E4M3, "%s o=%d" % (shape, o))


@pytest.mark.parametrize("dist", synth.DISTRIBUTIONS)
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_value_distributions(dist, dtype, elem):
    x = as_dtype(synth.draw(dist, (256, 640), synth.seed_for(5, synth.DISTRIBUTIONS.index(dist))), dtype)
    for rule in (orc.RULE_PAPER, orc.RULE_OCP):
        check(x, dtype, BOTH, rule, elem, "%s rule=%d" % (dist, rule))


def test_extreme_magnitudes_keep_exact_scales():
    # blocks whose scale byte is 0 (X = 2^-127), 1, 254: the decoded product must stay exact
    x = np.zeros((64, 128), np.float32)
    x[0:32, 0:32] = np.float32(2.0 ** -140)
    x[0:32, 32:64] = np.float32(2.0 ** -118) * np.linspace(0.1, 1, 32, dtype=np.float32)
    x[32:64, 0:32] = np.float32(3.0e38)
    x[32:64, 64:96] = np.float32(1.5 * 2.0 ** -126)
    for elem in (orc.E4M3, orc.E5M2):
        for rule in (orc.RULE_PAPER, orc.RULE_OCP):
            check(x, "fp32", BOTH, rule, elem, "extremes")
            check(synth.f32_to_bf16_bits(x), "bf16", BOTH, rule, elem, "extremes bf16")


def test_representable_input_is_a_fixed_point():
    # values already on the E4M3 grid of their block come back unchanged
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 0x7F, size=(64, 256), dtype=np.uint8)
    codes[:, ::32] = 0x7E                                   # every row block holds the format maximum
    vals = np.array([orc.fp8_decode(int(c), orc.E4M3) for c in range(0x7F)], np.float32)[codes]
    expo = rng.integers(-20, 20, size=(64, 8))
    x = (vals.reshape(64, 8, 32) * np.exp2(expo)[:, :, None]).astype(np.float32).reshape(64, 256)
    got = gpu_fake_quantize(x, "fp32", ROW, orc.RULE_PAPER, orc.E4M3)
    assert np.array_equal(got["row"], x)


def test_idempotent():
    x = synth.f32_to_bf16_bits(synth.student_t((128, 512), 77))
    once = gpu_fake_quantize(x, "bf16", ROW, orc.RULE_PAPER, orc.E4M3)["row"]
    twice = gpu_fake_quantize(np.ascontiguousarray(once), "bf16", ROW, orc.RULE_PAPER, orc.E4M3)["row"]
    assert np.array_equal(once, twice)


def test_equals_quantize_then_dequantize_on_device():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.from_numpy(synth.f32_to_bf16_bits(synth.gradient_like((512, 1024), 9)).view(np.int16)).cuda().view(torch.bfloat16)
    for o in (B.ROW, B.COL):
        q, s, _, _ = B.alloc_quantize_outputs(512, 1024, o, B.SF_LINEAR) if o == B.ROW else (None, None, None, None)
        if o == B.COL:
            _, _, q, s = B.alloc_quantize_outputs(512, 1024, o, B.SF_LINEAR)
        B.mxfp8_quantize(x, o, B.RULE_PAPER, B.E4M3, q if o == B.ROW else None, s if o == B.ROW else None,
                         q if o == B.COL else None, s if o == B.COL else None, B.SF_LINEAR)
        back = torch.empty_like(x)
        B.mxfp8_dequantize(q, s, o, B.E4M3, B.SF_LINEAR, back)
        fq = torch.empty_like(x)
        B.mxfp8_fake_quantize(x, o, B.RULE_PAPER, B.E4M3, fq if o == B.ROW else None, fq if o == B.COL else None)
        torch.cuda.synchronize()
        assert torch.equal(back.view(torch.int16), fq.view(torch.int16))


def test_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 40, dtype=torch.bfloat16, device="cuda")       # cols % 16 != 0
    d = torch.empty_like(x)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_fake_quantize(x, B.COL, B.RULE_PAPER, B.E4M3, None, d)
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_fake_quantize(x, B.ROW, B.RULE_PAPER, B.E4M3, None, None)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_fake_quantize(x, B.ROW, 7, B.E4M3, torch.empty_like(x), None)


def test_paper_rule_keeps_block_maximum_ocp_rule_clips_it():
    # Sec. 3.1 / Appendix A.1: rounding the scale exponent up keeps amax/X inside the E4M3 range, so
    # the block maximum is only rounded (relative error <= 2^-4); the floor-based rule lets blocks with
    # amax/X in (448, 512) saturate, which clips their maximum by up to 12.5 %.
    x = synth.gaussian((1024, 2048), 2026)
    blocks = np.abs(x).reshape(1024, 64, 32)
    arg = blocks.argmax(axis=2)
    amax = np.take_along_axis(blocks, arg[:, :, None], axis=2)[:, :, 0].astype(np.float64)
    rel = {}
    for rule in (orc.RULE_PAPER, orc.RULE_OCP):
        fq = np.abs(gpu_fake_quantize(x, "fp32", ROW, rule, orc.E4M3)["row"]).reshape(1024, 64, 32)
        back = np.take_along_axis(fq, arg[:, :, None], axis=2)[:, :, 0].astype(np.float64)
        rel[rule] = np.abs(back - amax) / amax
        assert (back <= amax * (1 + 2.0 ** -4)).all()
    assert rel[orc.RULE_PAPER].max() <= 2.0 ** -4
    clipped = rel[orc.RULE_OCP] > 2.0 ** -4
    assert clipped.any() and rel[orc.RULE_OCP].max() <= 0.125
    # the clipped value is 1.75 * 2^floor(log2 amax), so the error passes 2^-4 once amax = m * 2^e has m > 1.75 / (1 - 2^-4)
    mant = amax / np.exp2(np.floor(np.log2(amax)))
    assert np.array_equal(clipped, mant > 1.75 / (1 - 2.0 ** -4))
