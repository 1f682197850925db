"""The 6- and 4-bit element formats of Table 1 (MXFP6: E2M3, E3M2; MXFP4: E2M1) through
mxfp8_quantize / mxfp8_quantize_multi / mxfp8_dequantize / mxfp8_fake_quantize: bit-exact
against the oracle, same scale algorithm as MXFP8."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import check_against_oracle
from test_fake_quant_gpu import check as check_round_trip

pytestmark = pytest.mark.gpu

ROW, COL, BOTH = 1, 2, 3
LINEAR, SWIZZLED = 0, 1
ELEMS = [orc.E2M3, orc.E3M2, orc.E2M1]


def as_dtype(x32, dtype):
    return synth.f32_to_bf16_bits(x32) if dtype == "bf16" else x32


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("rule", [orc.RULE_PAPER, orc.RULE_OCP])
@pytest.mark.parametrize("elem", ELEMS)
def test_pr1_reference_tensor(dtype, rule, elem):
    x = as_dtype(synth.pr1_tensor(0), dtype)
    for orientation in (ROW, COL, BOTH):
        check_against_oracle(x, dtype, orientation, rule, elem, SWIZZLED, "pr1 o=%d" % orientation)
    check_against_oracle(x, dtype, BOTH, rule, elem, LINEAR, "pr1 linear")


@pytest.mark.parametrize("dist", synth.DISTRIBUTIONS)
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("elem", ELEMS)
def test_value_distributions(dist, dtype, elem):
    # "nonfinite" includes NaN and +-Inf elements: these formats have no such codes (NaN -> +max, Inf -> +-max)
    x = as_dtype(synth.draw(dist, (256, 1024), synth.seed_for(6, synth.DISTRIBUTIONS.index(dist))), dtype)
    for rule in (orc.RULE_PAPER, orc.RULE_OCP):
        check_against_oracle(x, dtype, BOTH, rule, elem, SWIZZLED, "%s rule=%d" % (dist, rule))


@pytest.mark.parametrize("shape", [(32, 32), (7, 64), (160, 352), (384, 2080), (64, 48), (96, 16)])
@pytest.mark.parametrize("elem", ELEMS)
def test_ragged_shapes(shape, elem):
    rows, cols = shape
    for dtype in ("fp32", "bf16"):
        x = as_dtype(synth.student_t(shape, 77 + rows + cols), dtype)
        orients = ([ROW] if cols % 32 == 0 else []) + ([COL] if rows % 32 == 0 else [])
        if cols % 32 == 0 and rows % 32 == 0:
            orients.append(BOTH)
        for o in orients:
            check_against_oracle(x, dtype, o, orc.RULE_PAPER, elem, SWIZZLED, "%s o=%d" % (shape, o))


@pytest.mark.parametrize("elem", ELEMS)
def test_scale_boundaries_at_the_largest_normal(elem):
    # block maxima exactly at destmax * 2^k, one FP32 step above and below: the rule's rounding decides here
    top = {orc.E2M3: 7.5, orc.E3M2: 28.0, orc.E2M1: 6.0}[elem]
    x = np.zeros((96, 64), np.float32)
    k = np.arange(96) - 40
    x[:, 0] = np.float32(top) * np.exp2(k).astype(np.float32)
    x[:, 32] = np.nextafter(x[:, 0], np.float32(np.inf))
    x[:, 1] = np.float32(0.3) * x[:, 0]
    x[:, 33] = -np.nextafter(x[:, 0], np.float32(0))
    for rule in (orc.RULE_PAPER, orc.RULE_OCP):
        check_against_oracle(x, "fp32", BOTH, rule, elem, LINEAR, "boundaries")


@pytest.mark.parametrize("elem", ELEMS)
@pytest.mark.parametrize("dst", ["f32", "bf16"])
def test_dequantize_exhaustive_codes_and_scales(elem, dst):
    import torch
    from paper_2506_08027_b200 import binding as B
    bits = 4 if elem == orc.E2M1 else 6
    codes = (np.arange(256) % (1 << bits)).astype(np.uint8)
    q = np.tile(np.repeat(codes, 32)[None, :], (256, 1))            # [256, 8192]
    s = np.repeat(np.arange(256, dtype=np.uint8)[:, None], 256, axis=1)
    want = orc.dequantize(q, s, orc.ROW, elem, dst)
    out = torch.empty(q.shape, dtype=torch.float32 if dst == "f32" else torch.bfloat16, device="cuda")
    B.mxfp8_dequantize(torch.from_numpy(orc.pack_codes16(q, elem)).cuda(), torch.from_numpy(s).cuda().view(-1), B.ROW, elem,
                       B.SF_LINEAR, out)
    torch.cuda.synchronize()
    if dst == "f32":
        got = out.cpu().numpy()
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(got), nan)
        assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))
    else:
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        nan = (want & 0x7FFF) > 0x7F80
        assert np.array_equal((got & 0x7FFF) > 0x7F80, nan)
        assert np.array_equal(got[~nan], want[~nan])


@pytest.mark.parametrize("elem", ELEMS)
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_fake_quantize_round_trip(elem, dtype):
    for dist in ("gaussian", "gradient_like", "nonfinite"):
        x = as_dtype(synth.draw(dist, (160, 416), 31), dtype)
        for rule in (orc.RULE_PAPER, orc.RULE_OCP):
            check_round_trip(x, dtype, BOTH, rule, elem, "%s rule=%d" % (dist, rule))


def test_widths_that_do_not_fill_slots_are_unsupported():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 40, dtype=torch.bfloat16, device="cuda")           # 40 columns: no whole 16-code slots
    _, _, qc, sc = B.alloc_quantize_outputs(64, 40, B.COL, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error) as e:
        B.mxfp8_quantize(x, B.COL, B.RULE_PAPER, B.E2M3, None, None, qc, sc, B.SF_LINEAR)
    assert e.value.status == -5
    B.mxfp8_quantize(x, B.COL, B.RULE_PAPER, B.E4M3, None, None, qc, sc, B.SF_LINEAR)   # fine for 8-bit codes
    with pytest.raises(B.Mxfp8Error) as e:
        B.mxfp8_dequantize(qc, sc, B.COL, B.E2M1, B.SF_LINEAR, torch.empty(64, 40, device="cuda"))
    assert e.value.status == -5


MIXES = [(orc.E2M3, orc.E2M3), (orc.E3M2, orc.E3M2), (orc.E2M1, orc.E2M1), (orc.E2M3, orc.E4M3), (orc.E5M2, orc.E2M1),
         (orc.E3M2, orc.E2M1)]


@pytest.mark.parametrize("mix", MIXES)
@pytest.mark.parametrize("majors", ["kk", "km", "mm"])
def test_gemm_on_six_and_four_bit_operands(mix, majors):
    # mxfp8_quantize writes the operands (packed slots, swizzled scales), mxfp8_gemm multiplies them on the
    # tensor cores; the oracle quantizes and multiplies the same inputs in FP64
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import check_gemm_tolerance
    a_elem, b_elem = mix
    a_mn, b_mn = majors[0] == "m", majors[1] == "m"
    M, N, K = 384, 256, 512
    a = synth.gaussian((M, K), 3)
    b = synth.student_t((N, K), 4) * np.float32(0.1)

    def prep(x, elem, mn):
        stored = np.ascontiguousarray(x.T) if mn else x                     # MN-major: stored [K, MN], blocks run down K
        o = B.COL if mn else B.ROW
        outs = B.alloc_quantize_outputs(stored.shape[0], stored.shape[1], o, B.SF_SWIZZLED)
        B.mxfp8_quantize(torch.from_numpy(stored).cuda(), o, B.RULE_PAPER, elem, *outs, B.SF_SWIZZLED)
        q, s = (outs[2], outs[3]) if mn else (outs[0], outs[1])
        oq, os_ = orc.quantize(stored, orc.COL if mn else orc.ROW, orc.RULE_PAPER, elem)
        return q, s, oq, os_

    qa, sa, oqa, osa = prep(a, a_elem, a_mn)
    qb, sb, oqb, osb = prep(b, b_elem, b_mn)
    D = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.mxfp8_gemm(qa, sa, qb, sb, M, N, K, B.MN_MAJOR if a_mn else B.K_MAJOR, B.MN_MAJOR if b_mn else B.K_MAJOR, a_elem, b_elem, D)
    assert B.mxfp8_device_status() == 0
    d64, sabs = orc.gemm_f64(oqa, osa, oqb, osb, "mn" if a_mn else "k", "mn" if b_mn else "k", a_elem, b_elem)
    check_gemm_tolerance(D.cpu().numpy(), d64, sabs, "%s %s" % (mix, majors))


def test_gemm_rejects_unknown_element_codes_and_sub_byte_fused_output():
    import torch
    from paper_2506_08027_b200 import binding as B
    z = torch.zeros(128, 128, dtype=torch.uint8, device="cuda")
    sc = torch.zeros(512, dtype=torch.uint8, device="cuda")
    D = torch.empty(128, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(B.Mxfp8Error) as e:
        B.mxfp8_gemm(z, sc, z, sc, 128, 128, 128, B.K_MAJOR, B.K_MAJOR, 2, B.E4M3, D)     # 2 is no element code
    assert e.value.status == -2
    epi = B.make_epilogue(B.ROW, B.RULE_PAPER, B.E2M3, z, sc)
    with pytest.raises(B.Mxfp8Error) as e:
        B.mxfp8_gemm(z, sc, z, sc, 128, 128, 128, B.K_MAJOR, B.K_MAJOR, B.E4M3, B.E4M3, D, epi=epi)
    assert e.value.status == -5


@pytest.mark.parametrize("elem", ELEMS)
def test_batched_and_fused_conversions_take_the_small_formats(elem):
    # the batched launch, the activation prologue and the gated prologue with 6- / 4-bit elements: same results as the
    # plain conversion of the corresponding tensor (which the tests above check against the oracle)
    import torch
    from paper_2506_08027_b200 import binding as B
    S = B.SF_SWIZZLED
    xs = [synth.device_tensor("gaussian", shp, 70 + i) for i, shp in enumerate(((256, 512), (160, 352)))]
    single = [B.alloc_quantize_outputs(t.shape[0], t.shape[1], B.BOTH, S) for t in xs]
    multi = [B.alloc_quantize_outputs(t.shape[0], t.shape[1], B.BOTH, S) for t in xs]
    for t, o in zip(xs, single):
        B.mxfp8_quantize(t, B.BOTH, B.RULE_PAPER, elem, *o, S)
    B.mxfp8_quantize_multi(B.make_quantize_items([(t,) + o for t, o in zip(xs, multi)]), B.BF16, B.BOTH, B.RULE_PAPER, elem, S)
    torch.cuda.synchronize()
    for a, b in zip(single, multi):
        for u, v in zip(a, b):
            assert torch.equal(u, v)
    # relu ahead of the conversion == conversion of relu(x)
    x = xs[0]
    want = B.alloc_quantize_outputs(256, 512, B.BOTH, S)
    got = B.alloc_quantize_outputs(256, 512, B.BOTH, S)
    B.mxfp8_quantize(torch.relu(x).contiguous(), B.BOTH, B.RULE_PAPER, elem, *want, S)
    B.mxfp8_act_quantize(x, B.ACT_RELU, B.BOTH, B.RULE_PAPER, elem, *got, S)
    # relu(gate) * up == conversion of the BF16 product (FP32 product rounded once, as torch does for BF16 operands)
    g2 = synth.device_tensor("gaussian", (256, 2 * 512), 75)
    y = (torch.relu(g2[:, :512].float()) * g2[:, 512:].float()).to(torch.bfloat16).contiguous()
    want2 = B.alloc_quantize_outputs(256, 512, B.BOTH, S)
    got2 = B.alloc_quantize_outputs(256, 512, B.BOTH, S)
    B.mxfp8_quantize(y, B.BOTH, B.RULE_PAPER, elem, *want2, S)
    B.mxfp8_glu_quantize(g2, B.ACT_RELU, B.BOTH, B.RULE_PAPER, elem, *got2, S)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for a, b in ((want, got), (want2, got2)):
        for u, v in zip(a, b):
            assert torch.equal(u, v)
