"""The linear-layer step (Sec. 3.2: FPROP, DGRAD, WGRAD on MXFP8 copies quantized along each GEMM's
reduction axis) through mxfp8_linear / mxfp8_linear_host, against the oracle chain and against the
product of fake-quantized operands."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth

pytestmark = pytest.mark.gpu


def to_dev_bf16(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def from_dev_bf16(t):
    import torch
    return orc.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))


def oracle_linear(x, w, dy, rule):
    """FP64 results and |a||b| sums of the three GEMMs on the oracle's MXFP8 copies."""
    q = {}
    for name, t in (("x", x), ("w", w), ("dy", dy)):
        q[name] = {o: orc.quantize(t, o, rule, orc.E4M3) for o in (orc.ROW, orc.COL)}
    R, C = orc.ROW, orc.COL
    y = orc.gemm_f64(q["x"][R][0], q["x"][R][1], q["w"][R][0], q["w"][R][1], "k", "k")
    dx = orc.gemm_f64(q["dy"][R][0], q["dy"][R][1], q["w"][C][0], q["w"][C][1], "k", "mn")
    dw = orc.gemm_f64(q["dy"][C][0], q["dy"][C][1], q["x"][C][0], q["x"][C][1], "mn", "mn")
    return y, dx, dw


def check_bf16_result(got_f32, d64, sabs, what):
    # FP32 accumulation bound of the GEMM plus one BF16 rounding (8-bit significand: half an ulp <= 2^-8 relative)
    err = np.abs(got_f32.astype(np.float64) - d64)
    bound = 2.0 ** -16 * sabs + 2.0 ** -8 * np.abs(d64) + 2.0 ** -126
    worst = float((err / bound).max())
    assert worst <= 1.0, "%s: worst err/bound %.3g" % (what, worst)


def inputs(T, H, F, seed):
    x = synth.f32_to_bf16_bits(synth.gaussian((T, H), seed))
    w = synth.f32_to_bf16_bits(0.02 * synth.gaussian((F, H), seed + 1))
    dy = synth.f32_to_bf16_bits(synth.output_gradient((T, F), seed + 2))
    return x, w, dy


@pytest.mark.parametrize("shape", [(256, 384, 128), (128, 128, 640)])
@pytest.mark.parametrize("rule", [orc.RULE_PAPER, orc.RULE_OCP])
def test_linear_device_matches_oracle_chain(shape, rule):
    import torch
    from paper_2506_08027_b200 import binding as B
    T, H, F = shape
    xb, wb, dyb = inputs(T, H, F, 31 + T)
    x, w, dy = to_dev_bf16(xb), to_dev_bf16(wb), to_dev_bf16(dyb)
    y = torch.empty(T, F, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(T, H, dtype=torch.bfloat16, device="cuda")
    dw = torch.empty(F, H, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.mxfp8_linear_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
    before = B.mxfp8_launch_count()
    B.mxfp8_linear(x, w, dy, rule, y, dx, dw, ws)
    assert B.mxfp8_device_status() == 0
    assert B.mxfp8_launch_count() - before == 2        # one batched cast + one launch over the three GEMMs
    want = oracle_linear(orc.bf16_bits_to_f32(xb), orc.bf16_bits_to_f32(wb), orc.bf16_bits_to_f32(dyb), rule)
    for got, (d64, sabs), name in zip((y, dx, dw), want, ("fprop", "dgrad", "wgrad")):
        check_bf16_result(from_dev_bf16(got), d64, sabs, name)


@pytest.mark.parametrize("shape", [(256, 256, 384), (512, 128, 128), (1024, 384, 640), (2048, 512, 1152), (512, 256, 1024), (384, 128, 512), (1024, 256, 2048)])
def test_linear_host_equals_device_variant(shape):
    """T = 256 goes through in one piece; multiples of 512 tokens go through in four row chunks whose copies overlap."""
    import torch
    from paper_2506_08027_b200 import binding as B
    T, H, F = shape
    xb, wb, dyb = inputs(T, H, F, 77)
    x, w, dy = to_dev_bf16(xb), to_dev_bf16(wb), to_dev_bf16(dyb)
    outs = [torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in ((T, F), (T, H), (F, H))]
    ws = torch.empty(B.mxfp8_linear_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
    B.mxfp8_linear(x, w, dy, B.RULE_PAPER, outs[0], outs[1], outs[2], ws)
    hx, hw, hdy = (t.cpu().pin_memory() for t in (x, w, dy))
    houts = [torch.empty(o.shape, dtype=torch.bfloat16).pin_memory() for o in outs]
    hws = torch.empty(B.mxfp8_linear_host_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
    B.mxfp8_linear_host(hx, hw, hdy, B.RULE_PAPER, houts[0], houts[1], houts[2], hws)
    torch.cuda.synchronize()
    for d, h in zip(outs, houts):
        assert torch.equal(d.cpu().view(torch.int16), h.view(torch.int16))


def test_gemm_equals_product_of_fake_quantized_operands():
    # Sec. 3.1: an MXFP8 GEMM computes the product of the decoded (fake-quantized) operands;
    # the decoded values come from the fake-quantize kernel, the product is taken in FP64 on the host.
    import torch
    from paper_2506_08027_b200 import binding as B
    T, H, F = 256, 512, 384
    xb, wb, _ = inputs(T, H, F, 5)
    x, w = to_dev_bf16(xb), to_dev_bf16(wb)
    fx, fw = torch.empty_like(x), torch.empty_like(w)
    B.mxfp8_fake_quantize(x, B.ROW, B.RULE_PAPER, B.E4M3, fx, None)
    B.mxfp8_fake_quantize(w, B.ROW, B.RULE_PAPER, B.E4M3, fw, None)
    a64, b64 = from_dev_bf16(fx).astype(np.float64), from_dev_bf16(fw).astype(np.float64)
    d64, sabs = a64 @ b64.T, np.abs(a64) @ np.abs(b64).T
    qx, sx, _, _ = B.alloc_quantize_outputs(T, H, B.ROW, B.SF_SWIZZLED)
    qw, sw, _, _ = B.alloc_quantize_outputs(F, H, B.ROW, B.SF_SWIZZLED)
    B.mxfp8_quantize(x, B.ROW, B.RULE_PAPER, B.E4M3, qx, sx, None, None, B.SF_SWIZZLED)
    B.mxfp8_quantize(w, B.ROW, B.RULE_PAPER, B.E4M3, qw, sw, None, None, B.SF_SWIZZLED)
    D = torch.empty(T, F, dtype=torch.float32, device="cuda")
    B.mxfp8_gemm(qx, sx, qw, sw, T, F, H, B.K_MAJOR, B.K_MAJOR, B.E4M3, B.E4M3, D)
    assert B.mxfp8_device_status() == 0
    err = np.abs(D.cpu().numpy().astype(np.float64) - d64)
    assert (err <= 2.0 ** -16 * sabs + 2.0 ** -126).all()
    assert np.sqrt((err ** 2).sum()) <= 1e-5 * np.sqrt((d64 ** 2).sum())


def test_linear_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    T, H, F = 128, 128, 128
    ws = torch.empty(B.mxfp8_linear_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.Mxfp8Error):        # workspace too small
        B.mxfp8_linear(z(T, H), z(F, H), z(T, F), B.RULE_PAPER, z(T, F), z(T, H), z(F, H), ws[:1024])
    with pytest.raises(B.Mxfp8Error):        # T not a multiple of 128
        B.mxfp8_linear(z(96, H), z(F, H), z(96, F), B.RULE_PAPER, z(96, F), z(96, H), z(F, H), ws)
    with pytest.raises(B.Mxfp8Error):        # unknown rule
        B.mxfp8_linear(z(T, H), z(F, H), z(T, F), 9, z(T, F), z(T, H), z(F, H), ws)
    assert B.mxfp8_linear_ws_bytes(0, 1, 1) == 0


def test_linear_step_can_be_captured_in_a_cuda_graph():
    # the device-pointer entry points only enqueue work on the caller's stream (no allocation, no synchronisation),
    # so a step can be captured once and replayed: replay on new inputs must equal the eager call bit for bit
    import torch
    from paper_2506_08027_b200 import binding as B
    T, H, F = 512, 256, 384
    xb, wb, dyb = inputs(T, H, F, 11)
    x, w, dy = to_dev_bf16(xb), to_dev_bf16(wb), to_dev_bf16(dyb)
    outs = [torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in ((T, F), (T, H), (F, H))]
    ws = torch.empty(B.mxfp8_linear_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
    B.mxfp8_linear(x, w, dy, B.RULE_PAPER, *outs, ws)                 # first use outside the capture (kernel attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.mxfp8_linear(x, w, dy, B.RULE_PAPER, *outs, ws)
    # new inputs into the captured buffers, replay, and compare with an eager call on copies
    xb2, wb2, dyb2 = inputs(T, H, F, 12)
    x.copy_(to_dev_bf16(xb2)); w.copy_(to_dev_bf16(wb2)); dy.copy_(to_dev_bf16(dyb2))
    for o in outs:
        o.zero_()
    launches = B.mxfp8_launch_count()
    graph.replay()
    torch.cuda.synchronize()
    assert B.mxfp8_launch_count() == launches                          # nothing went through the host entry points
    replayed = [o.clone() for o in outs]
    eager = [torch.empty_like(o) for o in outs]
    ws2 = torch.empty_like(ws)
    B.mxfp8_linear(x, w, dy, B.RULE_PAPER, *eager, ws2)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for a, b in zip(replayed, eager):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        assert a.float().abs().sum() > 0
