"""mxfp8_act_grad_quantize: the backward of an elementwise activation fused ahead of the conversion, dz = act'(z) * dh
(an activation gradient, converted like one: Sec. 3.2).  relu and squared relu are exact arithmetic: bit-exact against
the oracle.  silu and tanh-gelu use the device's fast FP32 exponential and division: almost every code equals the
oracle's, the rest differ by one code step at a rounding boundary, and the decoded error equals the oracle's."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import Guarded, logical_scales_from_swizzled, assert_q_equal

pytestmark = pytest.mark.gpu
ROW, COL, BOTH = 1, 2, 3


def as_dtype(x32, dtype):
    return synth.f32_to_bf16_bits(x32) if dtype == "bf16" else x32


def values(a, dtype):
    return orc.bf16_bits_to_f32(a) if dtype == "bf16" else a


def gpu_act_grad_quantize(dh_np, z_np, dtype, act, orientation, rule, elem):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = z_np.shape
    dev = (lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)) if dtype == "bf16" else (lambda a: torch.from_numpy(a).cuda())
    dh, z = dev(dh_np), dev(z_np)
    keep = (dh.clone(), z.clone())
    bufs, args = {}, []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            bufs[name] = (Guarded(rows * cols), Guarded(B.mxfp8_scale_bytes(rows, cols, o, B.SF_SWIZZLED)))
            args += [bufs[name][0].view.view(rows, cols), bufs[name][1].view]
        else:
            args += [None, None]
    before = B.mxfp8_launch_count()
    B.mxfp8_act_grad_quantize(dh, z, act, orientation, rule, elem, *args, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0 and B.mxfp8_launch_count() - before == 1
    assert torch.equal(dh.view(torch.uint8), keep[0].view(torch.uint8)) and torch.equal(z.view(torch.uint8), keep[1].view(torch.uint8))   # inputs untouched
    out = {}
    for name, (q, s) in bufs.items():
        q.check(); s.check()
        mn, nkb = (rows, cols // 32) if name == "row" else (cols, rows // 32)
        logical = logical_scales_from_swizzled(s.numpy(), mn, nkb)
        out[name] = (orc.unpack_codes16(q.numpy().reshape(rows, cols), elem), logical if name == "row" else np.ascontiguousarray(logical.T))
    return out


def oracle_grad_then_quantize(dh, z, dtype, act, o, rule, elem):
    y = orc.activation_grad(values(z, dtype), values(dh, dtype), act, "bf16" if dtype == "bf16" else "f32")
    y = orc.bf16_bits_to_f32(y) if dtype == "bf16" else y
    return (y,) + tuple(orc.quantize(y, o, rule, elem))


@pytest.mark.parametrize("act", [orc.ACT_RELU, orc.ACT_RELU2])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2, orc.E2M1])
def test_exact_activation_gradients_bit_exact(act, dtype, elem):
    for shape in ((256, 640), (160, 352), (96, 4096 + 128), (33 * 32, 96)):
        z = as_dtype(synth.gaussian(shape, 21 + act) * np.float32(2.0), dtype)
        dh = as_dtype(synth.output_gradient(shape, 31 + act), dtype)
        got = gpu_act_grad_quantize(dh, z, dtype, act, BOTH, orc.RULE_PAPER, elem)
        for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
            _, wq, ws = oracle_grad_then_quantize(dh, z, dtype, act, o, orc.RULE_PAPER, elem)
            assert np.array_equal(got[name][1], ws), "scales %s %s" % (shape, name)
            assert_q_equal(got[name][0], wq, elem, "%s %s" % (shape, name))


def test_relu_gradient_passes_specials_of_dh_where_z_is_positive():
    z = np.ones((64, 64), np.float32)
    z[:, 1] = -1.0
    dh = synth.gaussian((64, 64), 5)
    dh[3, 0], dh[4, 0], dh[5, 0], dh[6, 1] = np.inf, -np.inf, np.nan, np.inf       # column 1 is masked: 0 * Inf = NaN, as in the oracle
    got = gpu_act_grad_quantize(dh, z, "fp32", orc.ACT_RELU, BOTH, orc.RULE_OCP, orc.E4M3)
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        _, wq, ws = oracle_grad_then_quantize(dh, z, "fp32", orc.ACT_RELU, o, orc.RULE_OCP, orc.E4M3)
        assert np.array_equal(got[name][1], ws)
        assert_q_equal(got[name][0], wq, orc.E4M3, name)
    assert got["row"][0][3, 0] == 0x7E and got["row"][0][4, 0] == 0xFE and (got["row"][0][5, 0] & 0x7F) == 0x7F


@pytest.mark.parametrize("act", [orc.ACT_SILU, orc.ACT_GELU_TANH])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_transcendental_gradients_match_up_to_rounding_boundaries(act, dtype):
    shape = (512, 1024)
    z = as_dtype(synth.gaussian(shape, 6) * np.float32(2.5), dtype)
    dh = as_dtype(synth.gaussian(shape, 7), dtype)
    got = gpu_act_grad_quantize(dh, z, dtype, act, BOTH, orc.RULE_PAPER, orc.E4M3)
    for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
        y, wq, ws = oracle_grad_then_quantize(dh, z, dtype, act, o, orc.RULE_PAPER, orc.E4M3)
        gq, gs = got[name]
        same_scale = gs == ws
        assert same_scale.mean() >= 0.999
        blk = np.repeat(same_scale, 32, axis=1) if o == orc.ROW else np.repeat(same_scale, 32, axis=0)
        diff = (gq != wq) & blk
        assert diff.mean() <= 3e-3, "too many codes differ: %.2e" % diff.mean()
        a, b = gq[diff].astype(np.int32), wq[diff].astype(np.int32)
        assert (np.abs((a & 0x7F) - (b & 0x7F)) <= 1).all()
        d_gpu = orc.dequantize_f64(gq, gs, o, orc.E4M3)
        d_orc = orc.dequantize_f64(wq, ws, o, orc.E4M3)
        assert np.sqrt(((d_gpu - y) ** 2).sum()) <= 1.001 * np.sqrt(((d_orc - y) ** 2).sum())


@pytest.mark.parametrize("shape", [(1024, 2048), (8192, 4096 + 128)])   # the second: tiles handed out by the stream's counter, ragged last tile
def test_equals_separate_gradient_then_quantize_on_device(shape):
    import torch
    from paper_2506_08027_b200 import binding as B
    z = synth.device_tensor("activation", shape, 9)
    dh = synth.device_tensor("output_gradient", shape, 10)
    y = (torch.where(z.float() > 0, 2.0 * z.float(), torch.zeros((), device="cuda")) * dh.float()).to(torch.bfloat16)
    a = B.alloc_quantize_outputs(*shape, B.BOTH, B.SF_SWIZZLED)
    b = B.alloc_quantize_outputs(*shape, B.BOTH, B.SF_SWIZZLED)
    for t in a + b:
        t.zero_()
    B.mxfp8_act_grad_quantize(dh, z, B.ACT_RELU2, B.BOTH, B.RULE_PAPER, B.E4M3, *a, B.SF_SWIZZLED)
    B.mxfp8_quantize(y, B.BOTH, B.RULE_PAPER, B.E4M3, *b, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for u, v in zip(a, b):
        assert torch.equal(u, v)


def test_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    q, s, _, _ = B.alloc_quantize_outputs(64, 64, B.ROW, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_act_grad_quantize(x, x, B.ACT_NONE, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)   # no derivative to apply
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_act_grad_quantize(x, x, 9, B.ROW, B.RULE_PAPER, B.E4M3, q, s, None, None, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):
        B.mxfp8_act_grad_quantize(x, x, B.ACT_RELU, B.ROW, B.RULE_PAPER, B.E4M3, q, None, None, None, B.SF_LINEAR)
    assert B.lib().mxfp8_act_grad_quantize(None, x.data_ptr(), B.BF16, 64, 64, B.ACT_RELU, B.ROW, B.RULE_PAPER, B.E4M3, q.data_ptr(), s.data_ptr(),
                                           None, None, B.SF_LINEAR, None) == B.ERR_NULL
