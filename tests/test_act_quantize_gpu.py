"""mxfp8_act_quantize: an activation function fused ahead of the conversion (Sec. 3.2 keeps the activation in
high precision and converts its result).  relu and squared relu are exact arithmetic: bit-exact against the oracle.
silu and tanh-gelu use the device's FP32 exp / tanh: almost every code equals the oracle's, the rest differ by one
code step at a rounding boundary, and the decoded result stays within the format's error of the FP64 activation."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import Guarded, logical_scales_from_swizzled, assert_q_equal

pytestmark = pytest.mark.gpu

ROW, COL, BOTH = 1, 2, 3


def gpu_act_quantize(src_np, dtype, act, orientation, rule, elem):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = src_np.shape
    src = torch.from_numpy(src_np.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(src_np).cuda()
    bufs, args = {}, []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            bufs[name] = (Guarded(rows * cols), Guarded(B.mxfp8_scale_bytes(rows, cols, o, B.SF_SWIZZLED)))
            args += [bufs[name][0].view.view(rows, cols), bufs[name][1].view]
        else:
            args += [None, None]
    B.mxfp8_act_quantize(src, act, orientation, rule, elem, *args, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    out = {}
    for name, (q, s) in bufs.items():
        q.check(); s.check()
        mn, nkb = (rows, cols // 32) if name == "row" else (cols, rows // 32)
        logical = logical_scales_from_swizzled(s.numpy(), mn, nkb)
        out[name] = (orc.unpack_codes16(q.numpy().reshape(rows, cols), elem), logical if name == "row" else np.ascontiguousarray(logical.T))
    return out


def oracle_act_then_quantize(src_np, dtype, act, o, rule, elem):
    x = orc.bf16_bits_to_f32(src_np) if dtype == "bf16" else src_np
    y = orc.activation(x, act, "bf16" if dtype == "bf16" else "f32")
    y = orc.bf16_bits_to_f32(y) if dtype == "bf16" else y
    return (y,) + tuple(orc.quantize(y, o, rule, elem))


def as_dtype(x32, dtype):
    return synth.f32_to_bf16_bits(x32) if dtype == "bf16" else x32


@pytest.mark.parametrize("act", [orc.ACT_RELU, orc.ACT_RELU2, orc.ACT_NONE])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2, orc.E2M3])
def test_exact_activations_bit_exact(act, dtype, elem):
    for dist, shape in (("gaussian", (256, 640)), ("nonfinite", (160, 352)), ("gradient_like", (96, 4096 + 128))):
        x = as_dtype(synth.draw(dist, shape, 11 + act), dtype)
        got = gpu_act_quantize(x, dtype, act, BOTH, orc.RULE_PAPER, elem)
        for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
            _, wq, ws = oracle_act_then_quantize(x, dtype, act, o, orc.RULE_PAPER, elem)
            assert np.array_equal(got[name][1], ws), "scales %s %s" % (dist, name)
            assert_q_equal(got[name][0], wq, elem, "%s %s" % (dist, name))


def test_squared_relu_overflow_and_ocp_rule():
    # squares that overflow FP32 / BF16 become Inf and saturate to the largest code; the scale ignores them
    x = np.zeros((64, 64), np.float32)
    x[:, 0] = 1.0e20
    x[:, 1] = 3.0
    x[:, 2] = -5.0
    x[:, 33] = 2.0 ** -70
    for dtype in ("fp32", "bf16"):
        xs = as_dtype(x, dtype)
        got = gpu_act_quantize(xs, dtype, orc.ACT_RELU2, BOTH, orc.RULE_OCP, orc.E4M3)
        for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
            _, wq, ws = oracle_act_then_quantize(xs, dtype, orc.ACT_RELU2, o, orc.RULE_OCP, orc.E4M3)
            assert np.array_equal(got[name][1], ws)
            assert_q_equal(got[name][0], wq, orc.E4M3, name)
        assert (got["row"][0][:, 0] == 0x7E).all()


@pytest.mark.parametrize("act", [orc.ACT_SILU, orc.ACT_GELU_TANH])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_transcendental_activations_match_up_to_rounding_boundaries(act, dtype):
    x = as_dtype(synth.gaussian((512, 1024), 5) * np.float32(2.5), dtype)
    got = gpu_act_quantize(x, dtype, act, BOTH, orc.RULE_PAPER, orc.E4M3)
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        y, wq, ws = oracle_act_then_quantize(x, dtype, act, o, orc.RULE_PAPER, orc.E4M3)
        gq, gs = got[name]
        # a block's scale can move only if its amax sat on a power-of-two boundary: rare
        same_scale = gs == ws
        assert same_scale.mean() >= 0.999
        blk = np.repeat(same_scale, 32, axis=1) if o == orc.ROW else np.repeat(same_scale, 32, axis=0)
        diff = (gq != wq) & blk
        assert diff.mean() <= 2e-3, "too many codes differ: %.2e" % diff.mean()
        # where a code differs it is the neighbouring code (same sign, magnitude code one apart)
        a, b = gq[diff].astype(np.int32), wq[diff].astype(np.int32)
        assert ((a & 0x80) == (b & 0x80))[(a & 0x7F > 0) & (b & 0x7F > 0)].all()
        assert (np.abs((a & 0x7F) - (b & 0x7F)) <= 1).all()
        # and the decoded tensor is as close to the FP64 activation as the oracle's own
        d_gpu = orc.dequantize_f64(gq, gs, o, orc.E4M3)
        d_orc = orc.dequantize_f64(wq, ws, o, orc.E4M3)
        err_gpu = np.sqrt(((d_gpu - y) ** 2).sum())
        err_orc = np.sqrt(((d_orc - y) ** 2).sum())
        assert err_gpu <= 1.001 * err_orc


@pytest.mark.parametrize("shape", [(1024, 2048), (8192, 4096 + 128)])   # the second: tiles handed out by the stream's counter, ragged last tile
def test_equals_separate_activation_then_quantize_on_device(shape):
    # the fused call against mxfp8_quantize applied to a tensor that holds relu(x)^2 (computed by torch in FP32)
    import torch
    from paper_2506_08027_b200 import binding as B
    x = synth.device_tensor("activation", shape, 9)
    y = (torch.relu(x.float()) ** 2).to(torch.bfloat16)
    a = B.alloc_quantize_outputs(*shape, B.BOTH, B.SF_SWIZZLED)
    b = B.alloc_quantize_outputs(*shape, B.BOTH, B.SF_SWIZZLED)
    for t in a + b:
        t.zero_()
    B.mxfp8_act_quantize(x, B.ACT_RELU2, B.BOTH, B.RULE_PAPER, B.E4M3, *a, B.SF_SWIZZLED)
    B.mxfp8_quantize(y, B.BOTH, B.RULE_PAPER, B.E4M3, *b, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    for u, v in zip(a, b):
        assert torch.equal(u, v)


def test_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    q, s, _, _ = B.alloc_quantize_outputs(64, 64, B.ROW, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_act_quantize(x, 9, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_act_quantize(x, B.ACT_RELU, B.ROW, B.RULE_PAPER, B.E4M3, q, None, None, None, B.SF_LINEAR)
    y = torch.zeros(64, 40, dtype=torch.bfloat16, device="cuda")
    _, _, qc, sc = B.alloc_quantize_outputs(64, 40, B.COL, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_act_quantize(y, B.ACT_RELU, B.COL, B.RULE_PAPER, B.E4M3, None, None, qc, sc, B.SF_LINEAR)


# ------------------------------------------------------------------------------------------ RMS normalisation

def gpu_rmsnorm_quantize(src_np, gamma_np, dtype, eps, orientation, elem=orc.E4M3):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = src_np.shape
    if dtype == "bf16":
        src = torch.from_numpy(src_np.view(np.int16)).cuda().view(torch.bfloat16)
        gamma = torch.from_numpy(gamma_np.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        src, gamma = torch.from_numpy(src_np).cuda(), torch.from_numpy(gamma_np).cuda()
    rstd = Guarded(rows * 4)
    bufs, args = {}, []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            bufs[name] = (Guarded(rows * cols), Guarded(B.mxfp8_scale_bytes(rows, cols, o, B.SF_SWIZZLED)))
            args += [bufs[name][0].view.view(rows, cols), bufs[name][1].view]
        else:
            args += [None, None]
    before = B.mxfp8_launch_count()
    B.mxfp8_rmsnorm_quantize(src, gamma, eps, rstd.view.view(torch.float32), orientation, B.RULE_PAPER, elem, *args, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0 and B.mxfp8_launch_count() - before == 2
    rstd.check()
    out = {"rstd": rstd.numpy().view(np.float32).copy()}
    for name, (q, s) in bufs.items():
        q.check(); s.check()
        mn, nkb = (rows, cols // 32) if name == "row" else (cols, rows // 32)
        logical = logical_scales_from_swizzled(s.numpy(), mn, nkb)
        out[name] = (orc.unpack_codes16(q.numpy().reshape(rows, cols), elem), logical if name == "row" else np.ascontiguousarray(logical.T))
    return out


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", [(256, 512), (160, 352), (96, 4096 + 128), (32, 2048)])
def test_rmsnorm_quantize(dtype, shape):
    rows, cols = shape
    x32 = synth.gaussian(shape, 3 + rows) * np.exp2(np.random.default_rng(rows).integers(-6, 6, (rows, 1))).astype(np.float32)
    g32 = (1.0 + 0.2 * synth.gaussian((1, cols), 4)[0]).astype(np.float32)
    x, g = as_dtype(x32, dtype), as_dtype(g32, dtype)
    xv = orc.bf16_bits_to_f32(x) if dtype == "bf16" else x
    gv = orc.bf16_bits_to_f32(g) if dtype == "bf16" else g
    got = gpu_rmsnorm_quantize(x, g, dtype, 1e-5, BOTH)
    # the statistics: FP32 accumulation against the FP64 definition
    _, want_rstd = orc.rmsnorm(xv, gv, 1e-5)
    assert np.abs(got["rstd"] - want_rstd).max() <= 2.0 ** -20 * np.abs(want_rstd).max()
    # given those statistics everything after is exact arithmetic: bit-exact against the oracle
    y, _ = orc.rmsnorm(xv, gv, 1e-5, "bf16" if dtype == "bf16" else "f32", got["rstd"])
    y = orc.bf16_bits_to_f32(y) if dtype == "bf16" else y
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        wq, ws = orc.quantize(y, o, orc.RULE_PAPER, orc.E4M3)
        assert np.array_equal(got[name][1], ws), "scales %s" % name
        assert_q_equal(got[name][0], wq, orc.E4M3, name)


# ------------------------------------------------------------------------------------------ layer normalisation

def gpu_layernorm_quantize(src_np, gamma_np, beta_np, dtype, eps, orientation, elem=orc.E4M3):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = src_np.shape

    def dev(a):
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(a).cuda()
    src, gamma, beta = dev(src_np), dev(gamma_np), dev(beta_np)
    mean, rstd = Guarded(rows * 4), Guarded(rows * 4)
    bufs, args = {}, []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            bufs[name] = (Guarded(rows * cols), Guarded(B.mxfp8_scale_bytes(rows, cols, o, B.SF_SWIZZLED)))
            args += [bufs[name][0].view.view(rows, cols), bufs[name][1].view]
        else:
            args += [None, None]
    before = B.mxfp8_launch_count()
    B.mxfp8_layernorm_quantize(src, gamma, beta, eps, mean.view.view(torch.float32), rstd.view.view(torch.float32), orientation,
                               B.RULE_PAPER, elem, *args, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0 and B.mxfp8_launch_count() - before == 2
    mean.check(); rstd.check()
    out = {"mean": mean.numpy().view(np.float32).copy(), "rstd": rstd.numpy().view(np.float32).copy()}
    for name, (q, s) in bufs.items():
        q.check(); s.check()
        mn, nkb = (rows, cols // 32) if name == "row" else (cols, rows // 32)
        logical = logical_scales_from_swizzled(s.numpy(), mn, nkb)
        out[name] = (orc.unpack_codes16(q.numpy().reshape(rows, cols), elem), logical if name == "row" else np.ascontiguousarray(logical.T))
    return out


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", [(256, 512), (160, 352), (96, 4096 + 128), (32, 2048)])
def test_layernorm_quantize(dtype, shape):
    rows, cols = shape
    rng = np.random.default_rng(rows)
    x32 = (synth.gaussian(shape, 13 + rows) * np.exp2(rng.integers(-6, 6, (rows, 1))) + rng.standard_normal((rows, 1)) * 4).astype(np.float32)
    g32 = (1.0 + 0.2 * synth.gaussian((1, cols), 14)[0]).astype(np.float32)
    b32 = (0.3 * synth.gaussian((1, cols), 15)[0]).astype(np.float32)
    x, g, b = as_dtype(x32, dtype), as_dtype(g32, dtype), as_dtype(b32, dtype)
    val = (lambda a: orc.bf16_bits_to_f32(a)) if dtype == "bf16" else (lambda a: a)
    xv, gv, bv = val(x), val(g), val(b)
    got = gpu_layernorm_quantize(x, g, b, dtype, 1e-5, BOTH)
    # the statistics: FP32 accumulation against the FP64 definition
    _, want_mean, want_rstd = orc.layernorm(xv, gv, bv, 1e-5)
    assert np.abs(got["mean"] - want_mean).max() <= 2.0 ** -20 * np.abs(xv).max()
    assert np.abs(got["rstd"] - want_rstd).max() <= 2.0 ** -18 * np.abs(want_rstd).max()
    # given those statistics everything after is exact arithmetic: bit-exact against the oracle
    y, _, _ = orc.layernorm(xv, gv, bv, 1e-5, "bf16" if dtype == "bf16" else "f32", got["mean"], got["rstd"])
    y = orc.bf16_bits_to_f32(y) if dtype == "bf16" else y
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        wq, ws = orc.quantize(y, o, orc.RULE_PAPER, orc.E4M3)
        assert np.array_equal(got[name][1], ws), "scales %s" % name
        assert_q_equal(got[name][0], wq, orc.E4M3, name)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_layernorm_statistics_with_an_outlier_in_the_first_column(dtype):
    """The statistics pass sums around the row's first element; rows that begin with an outlier of 10^3 to 10^4
    standard deviations (and rows with the outlier elsewhere, or none) must still give the mean and rstd of the
    FP64 definition."""
    rows, cols = 96, 2048
    rng = np.random.default_rng(5)
    x32 = (synth.gaussian((rows, cols), 31) + rng.standard_normal((rows, 1)) * 3).astype(np.float32)
    x32[0:32, 0] += np.float32(1e3) * rng.choice([-1.0, 1.0], 32).astype(np.float32)
    x32[32:64, 0] += np.float32(1e4)
    x32[64:80, 777] -= np.float32(1e4)
    g32 = np.ones(cols, np.float32)
    b32 = np.zeros(cols, np.float32)
    x, g, b = as_dtype(x32, dtype), as_dtype(g32, dtype), as_dtype(b32, dtype)
    xv = orc.bf16_bits_to_f32(x) if dtype == "bf16" else x
    got = gpu_layernorm_quantize(x, g, b, dtype, 1e-5, ROW)
    _, want_mean, want_rstd = orc.layernorm(xv, g32, b32, 1e-5)
    assert np.abs(got["mean"] - want_mean).max() <= 2.0 ** -20 * np.abs(xv).max()
    assert (np.abs(got["rstd"] - want_rstd) <= 2.0 ** -18 * np.abs(want_rstd)).all()


def test_layernorm_equals_rmsnorm_on_centred_rows_without_bias():
    """Rows of small multiples of 1/4 in (v, -v) pairs and a zero bias: every sum the two statistics kernels form is exact,
    the mean is exactly zero, and the two normalisations are the same arithmetic."""
    rows, cols = 64, 256
    rng = np.random.default_rng(77)
    half = (rng.integers(1, 9, (rows, cols // 2)) * rng.choice([-1.0, 1.0], (rows, cols // 2)) / 4.0).astype(np.float32)   # no zeros: -0 + bias 0 = +0
    x = np.stack([half, -half], axis=2).reshape(rows, cols).copy()
    g = (1.0 + 0.2 * synth.gaussian((1, cols), 78)[0]).astype(np.float32)
    ln = gpu_layernorm_quantize(x, g, np.zeros(cols, np.float32), "fp32", 1e-5, BOTH)
    rms = gpu_rmsnorm_quantize(x, g, "fp32", 1e-5, BOTH)
    assert not ln["mean"].any()
    assert np.array_equal(ln["rstd"], rms["rstd"])
    for name in ("row", "col"):
        assert np.array_equal(ln[name][0], rms[name][0]) and np.array_equal(ln[name][1], rms[name][1])


def test_rmsnorm_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    g = torch.ones(64, dtype=torch.bfloat16, device="cuda")
    r = torch.empty(64, dtype=torch.float32, device="cuda")
    q, s, _, _ = B.alloc_quantize_outputs(64, 64, B.ROW, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_rmsnorm_quantize(x, g, -1.0, r, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_rmsnorm_quantize(x, g, 1e-5, r, B.COL, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
    # an all-zero row with eps = 0 has rstd = Inf and 0 * Inf = NaN elements: they become NaN codes, nothing faults
    B.mxfp8_rmsnorm_quantize(x, g, 0.0, r, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
    torch.cuda.synchronize()
    assert torch.isinf(r).all() and (q == 0x7F).all()


# ------------------------------------------------------------------------------------------ gated activation

def gpu_glu_quantize(src_np, dtype, act, orientation, elem=orc.E4M3):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, two_cols = src_np.shape
    cols = two_cols // 2
    src = torch.from_numpy(src_np.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(src_np).cuda()
    bufs, args = {}, []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            bufs[name] = (Guarded(rows * cols), Guarded(B.mxfp8_scale_bytes(rows, cols, o, B.SF_SWIZZLED)))
            args += [bufs[name][0].view.view(rows, cols), bufs[name][1].view]
        else:
            args += [None, None]
    B.mxfp8_glu_quantize(src, act, orientation, B.RULE_PAPER, elem, *args, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    out = {}
    for name, (q, s) in bufs.items():
        q.check(); s.check()
        mn, nkb = (rows, cols // 32) if name == "row" else (cols, rows // 32)
        logical = logical_scales_from_swizzled(s.numpy(), mn, nkb)
        out[name] = (orc.unpack_codes16(q.numpy().reshape(rows, cols), elem), logical if name == "row" else np.ascontiguousarray(logical.T))
    return out


@pytest.mark.parametrize("act", [orc.ACT_RELU, orc.ACT_NONE, orc.ACT_RELU2])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", [(256, 2 * 256), (160, 2 * 384), (96, 2 * 1408), (1056, 2 * 128)])
def test_gated_exact_activations_bit_exact(act, dtype, shape):
    # many tiles per CTA on the last shape: the up tile is prefetched one tile ahead
    x = as_dtype(synth.gaussian(shape, 21 + act + shape[0]) * np.float32(2.0), dtype)
    xv = orc.bf16_bits_to_f32(x) if dtype == "bf16" else x
    y = orc.glu(xv, act, "bf16" if dtype == "bf16" else "f32")
    y = orc.bf16_bits_to_f32(y) if dtype == "bf16" else y
    got = gpu_glu_quantize(x, dtype, act, BOTH)
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        wq, ws = orc.quantize(y, o, orc.RULE_PAPER, orc.E4M3)
        assert np.array_equal(got[name][1], ws), "scales %s" % name
        assert_q_equal(got[name][0], wq, orc.E4M3, name)


def test_swiglu_matches_up_to_rounding_boundaries_and_many_tiles():
    x = as_dtype(synth.gaussian((2048, 2 * 1408), 8) * np.float32(2.0), "bf16")         # 16 x 11 tiles on 296 CTAs? no: 176 tiles
    xv = orc.bf16_bits_to_f32(x)
    y = orc.bf16_bits_to_f32(orc.glu(xv, orc.ACT_SILU, "bf16"))
    got = gpu_glu_quantize(x, "bf16", orc.ACT_SILU, BOTH)
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        wq, ws = orc.quantize(y, o, orc.RULE_PAPER, orc.E4M3)
        gq, gs = got[name]
        same_scale = gs == ws
        assert same_scale.mean() >= 0.999
        blk = np.repeat(same_scale, 32, axis=1) if o == orc.ROW else np.repeat(same_scale, 32, axis=0)
        diff = (gq != wq) & blk
        assert diff.mean() <= 2e-3
        a, b = gq[diff].astype(np.int32), wq[diff].astype(np.int32)
        assert (np.abs((a & 0x7F) - (b & 0x7F)) <= 1).all()


def test_gated_equals_torch_reglu_then_quantize_on_device_large():
    # 8192 x (2 x 4096): more tiles than resident CTAs, every CTA walks several tiles
    import torch
    from paper_2506_08027_b200 import binding as B
    x = synth.device_tensor("activation", (8192, 2 * 4096), 12)
    xf = x.float()
    y = (torch.relu(xf[:, :4096]) * xf[:, 4096:]).to(torch.bfloat16).contiguous()
    a = B.alloc_quantize_outputs(8192, 4096, B.BOTH, B.SF_SWIZZLED)
    b = B.alloc_quantize_outputs(8192, 4096, B.BOTH, B.SF_SWIZZLED)
    for t in a + b:
        t.zero_()
    B.mxfp8_glu_quantize(x, B.ACT_RELU, B.BOTH, B.RULE_PAPER, B.E4M3, *a, B.SF_SWIZZLED)
    B.mxfp8_quantize(y, B.BOTH, B.RULE_PAPER, B.E4M3, *b, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for u, v in zip(a, b):
        assert torch.equal(u, v)


def test_gated_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 2 * 96, dtype=torch.bfloat16, device="cuda")          # 96 output columns: not whole tiles
    q, s, _, _ = B.alloc_quantize_outputs(64, 96, B.ROW, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error) as e:
        B.mxfp8_glu_quantize(x, B.ACT_SILU, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
    assert e.value.status == -5
    x = torch.zeros(64, 2 * 128, dtype=torch.bfloat16, device="cuda")
    q, s, _, _ = B.alloc_quantize_outputs(64, 128, B.ROW, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_glu_quantize(x, 11, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
