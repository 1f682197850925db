"""Parity of mxfp8_quantize / mxfp8_dequantize with the CPU oracle: bit-exact Q and scale bytes."""
import os
import struct

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import check_against_oracle, gpu_quantize, assert_q_equal

pytestmark = pytest.mark.gpu

ROW, COL, BOTH = 1, 2, 3
LINEAR, SWIZZLED = 0, 1


def as_dtype(x32, dtype):
    return synth.f32_to_bf16_bits(x32) if dtype == "bf16" else x32


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("rule", [orc.RULE_PAPER, orc.RULE_OCP])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_pr1_reference_tensor(dtype, rule, elem):
    # config 1: 256x512, row-scaled Gaussian with outliers, zero blocks, a block with amax 448
    x = as_dtype(synth.pr1_tensor(0), dtype)
    for orientation in (ROW, COL, BOTH):
        for layout in (LINEAR, SWIZZLED):
            check_against_oracle(x, dtype, orientation, rule, elem, layout, "pr1 o=%d l=%d" % (orientation, layout))


SHAPES = [(32, 32), (1, 32), (7, 64), (32, 128), (160, 352), (128, 128), (160, 416),
          (384, 8288), (96, 4096 + 128), (1024, 4096)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_shapes_and_ragged_tails(shape, dtype):
    rows, cols = shape
    x = as_dtype(synth.gaussian(shape, 1234 + rows + cols), dtype)
    orients = [ROW]
    if rows % 32 == 0:
        orients += [COL, BOTH]
    for o in orients:
        for layout in (LINEAR, SWIZZLED):
            check_against_oracle(x, dtype, o, orc.RULE_PAPER, orc.E4M3, layout, "%s o=%d l=%d" % (shape, o, layout))


@pytest.mark.parametrize("cols", [100, 33, 2, 130])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_column_blocks_with_odd_width(cols, dtype):
    x = as_dtype(synth.gaussian((64, cols), 99 + cols), dtype)
    for layout in (LINEAR, SWIZZLED):
        check_against_oracle(x, dtype, COL, orc.RULE_PAPER, orc.E4M3, layout, "cols=%d" % cols)


@pytest.mark.parametrize("dist", synth.DISTRIBUTIONS)
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
def test_distributions(dist, dtype, elem):
    x = as_dtype(synth.draw(dist, (256, 1024), synth.seed_for(4, synth.DISTRIBUTIONS.index(dist))), dtype)
    for rule in (orc.RULE_PAPER, orc.RULE_OCP):
        check_against_oracle(x, dtype, BOTH, rule, elem, SWIZZLED, dist)


def test_nonfinite_dense():
    # many NaN / Inf, including whole blocks of them, in both orientations
    rng = np.random.default_rng(5)
    x = synth.gaussian((128, 256), 77)
    pick = rng.random(x.shape)
    x[pick < 0.05] = np.nan
    x[(pick >= 0.05) & (pick < 0.10)] = np.inf
    x[(pick >= 0.10) & (pick < 0.15)] = -np.inf
    x[3, 32:64] = np.nan
    x[32:64, 9] = np.inf
    x[5, 64:96] = [np.inf, -np.inf] * 16
    for dtype in ("fp32", "bf16"):
        for elem in (orc.E4M3, orc.E5M2):
            check_against_oracle(as_dtype(x, dtype), dtype, BOTH, orc.RULE_PAPER, elem, LINEAR, "nonfinite")


def test_fp32_extremes_and_subnormals():
    # FP32 subnormal inputs are honoured; the largest finite inputs do not overflow the scale
    bits = np.array([0x00000001, 0x00000200, 0x00080000, 0x007FFFFF, 0x00800000, 0x03E00000, 0x04600000,
                     0x04600001, 0x07E00001, 0x7F7FFFFF, 0x7F000000, 0x80000000, 0x80000001], dtype=np.uint32)
    rng = np.random.default_rng(8)
    x = np.zeros((64, 128), dtype=np.float32)
    flat = x.reshape(-1)
    pos = rng.choice(flat.size, size=bits.size * 8, replace=False)
    flat[pos] = np.tile(bits, 8).view(np.float32)
    # plus blocks made only of subnormals
    x[10, 32:64] = np.frombuffer(struct.pack("<I", 0x00080000), np.float32)[0]
    for rule in (orc.RULE_PAPER, orc.RULE_OCP):
        for elem in (orc.E4M3, orc.E5M2):
            check_against_oracle(x, "fp32", BOTH, rule, elem, LINEAR, "extremes")


def test_handworked_blocks_on_gpu(golden_dir):
    from test_oracle_pins import read_golden, ELEMS
    rows_ = read_golden(os.path.join(golden_dir, "handworked_blocks.txt"))
    for elem_name in ("e4m3", "e5m2"):
        sel = [r for r in rows_ if r[0] == elem_name]
        x = np.zeros((32, 32 * len(sel)), dtype=np.float32)
        for i, r in enumerate(sel):
            x[0, 32 * i + 3] = np.frombuffer(struct.pack("<I", int(r[1], 16)), np.float32)[0]
        for rule, bi, qi in ((orc.RULE_PAPER, 2, 3), (orc.RULE_OCP, 4, 5)):
            got = gpu_quantize(x, "fp32", ROW, rule, ELEMS[elem_name], LINEAR)
            for i, r in enumerate(sel):
                assert got["s_row"][0, i] == int(r[bi], 16), r
                assert got["q_row"][0, 32 * i + 3] == int(r[qi], 16), r


def test_deterministic_and_both_equals_separate():
    x = synth.f32_to_bf16_bits(synth.gradient_like((512, 2048), 31))
    a = gpu_quantize(x, "bf16", BOTH, orc.RULE_PAPER, orc.E4M3, SWIZZLED)
    b = gpu_quantize(x, "bf16", BOTH, orc.RULE_PAPER, orc.E4M3, SWIZZLED)
    r = gpu_quantize(x, "bf16", ROW, orc.RULE_PAPER, orc.E4M3, SWIZZLED)
    c = gpu_quantize(x, "bf16", COL, orc.RULE_PAPER, orc.E4M3, SWIZZLED)
    for k in ("q_row", "q_col", "raw_s_row", "raw_s_col"):
        assert np.array_equal(a[k], b[k])
    assert np.array_equal(a["q_row"], r["q_row"]) and np.array_equal(a["raw_s_row"], r["raw_s_row"])
    assert np.array_equal(a["q_col"], c["q_col"]) and np.array_equal(a["raw_s_col"], c["raw_s_col"])


def test_large_tensor_sampled():
    # a benchmark-sized tensor (8192 x 8192 BF16, drawn on the device): the oracle checks a
    # strided sample of 128-row slabs plus the first and last slab
    import torch
    from paper_2506_08027_b200 import binding as B
    rows = cols = 8192
    src = synth.device_tensor("output_gradient", (rows, cols), synth.seed_for(2, 2))
    qr, sr, qc, sc = B.alloc_quantize_outputs(rows, cols, B.BOTH, B.SF_LINEAR)
    B.mxfp8_quantize(src, B.BOTH, B.RULE_PAPER, B.E4M3, qr, sr, qc, sc, B.SF_LINEAR)
    torch.cuda.synchronize()
    for r0 in (0, 1024 + 128, 4096 - 128, 8192 - 128):
        sl = slice(r0, r0 + 128)
        x = orc.bf16_bits_to_f32(src[sl].view(torch.int16).cpu().numpy().view(np.uint16))
        wq, ws = orc.quantize(x, orc.ROW)
        assert np.array_equal(sr.view(rows, cols // 32)[sl].cpu().numpy(), ws)
        assert_q_equal(qr[sl].cpu().numpy(), wq, orc.E4M3)
        wq, ws = orc.quantize(x, orc.COL)
        assert np.array_equal(sc.view(rows // 32, cols)[r0 // 32:r0 // 32 + 4].cpu().numpy(), ws)
        assert_q_equal(qc[sl].cpu().numpy(), wq, orc.E4M3)


def test_benchmark_step_cast_in_its_launch_configuration_sampled():
    # the benchmark's cast: X [8192, 2048], W [8192, 2048], dY [8192, 8192] (BF16, drawn on the device) in ONE
    # batched launch, both orientations, swizzled scales; the oracle checks sampled 128-row slabs of every tensor
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import logical_scales_from_swizzled
    T, H, F = 8192, 2048, 8192
    tensors = [synth.device_tensor("activation", (T, H), synth.seed_for(2, 0)),
               synth.device_tensor("weight", (F, H), synth.seed_for(2, 1)),
               synth.device_tensor("output_gradient", (T, F), synth.seed_for(2, 2))]
    outs = [B.alloc_quantize_outputs(t.shape[0], t.shape[1], B.BOTH, B.SF_SWIZZLED) for t in tensors]
    items = B.make_quantize_items([(t,) + o for t, o in zip(tensors, outs)])
    B.mxfp8_quantize_multi(items, B.BF16, B.BOTH, B.RULE_PAPER, B.E4M3, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for src, (qr, sr, qc, sc) in zip(tensors, outs):
        rows, cols = src.shape
        s_row = logical_scales_from_swizzled(sr.cpu().numpy(), rows, cols // 32)            # [rows, cols/32]
        s_col = logical_scales_from_swizzled(sc.cpu().numpy(), cols, rows // 32).T          # [rows/32, cols]
        for r0 in (0, 2048 + 128, rows - 128):
            sl = slice(r0, r0 + 128)
            x = orc.bf16_bits_to_f32(src[sl].view(torch.int16).cpu().numpy().view(np.uint16))
            wq, ws = orc.quantize(x, orc.ROW)
            assert np.array_equal(s_row[sl], ws)
            assert_q_equal(qr[sl].cpu().numpy(), wq, orc.E4M3)
            wq, ws = orc.quantize(x, orc.COL)
            assert np.array_equal(s_col[r0 // 32:r0 // 32 + 4], ws)
            assert_q_equal(qc[sl].cpu().numpy(), wq, orc.E4M3)


# ------------------------------------------------------------------------------- dequantize

@pytest.mark.parametrize("elem", [orc.E4M3, orc.E5M2])
@pytest.mark.parametrize("dst", ["f32", "bf16"])
def test_dequantize_exhaustive_codes_and_scales(elem, dst):
    import torch
    from paper_2506_08027_b200 import binding as B
    codes = np.arange(256, dtype=np.uint8)
    q = np.tile(np.repeat(codes, 32)[None, :], (256, 1))            # [256, 8192]
    s = np.repeat(np.arange(256, dtype=np.uint8)[:, None], 256, axis=1)
    want = orc.dequantize(q, s, orc.ROW, elem, dst)
    qd, sd = torch.from_numpy(q).cuda(), torch.from_numpy(s).cuda()
    out = torch.empty(q.shape, dtype=torch.float32 if dst == "f32" else torch.bfloat16, device="cuda")
    B.mxfp8_dequantize(qd, sd.view(-1), B.ROW, elem, B.SF_LINEAR, out)
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


@pytest.mark.parametrize("orientation", [ROW, COL])
@pytest.mark.parametrize("layout", [LINEAR, SWIZZLED])
@pytest.mark.parametrize("shape", [(256, 512), (96, 352), (64, 100)])
def test_dequantize_roundtrip_layouts(orientation, layout, shape):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = shape
    if orientation == ROW and cols % 32:
        pytest.skip("row blocks need cols % 32 == 0")
    x = synth.gradient_like(shape, 5 + rows)
    src = torch.from_numpy(x).cuda()
    outs = B.alloc_quantize_outputs(rows, cols, orientation, layout)
    B.mxfp8_quantize(src, orientation, B.RULE_PAPER, B.E4M3, *outs, layout)
    q, s = (outs[0], outs[1]) if orientation == ROW else (outs[2], outs[3])
    for dst_dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        dst = torch.empty(shape, dtype=dst_dtype, device="cuda")
        B.mxfp8_dequantize(q, s, orientation, B.E4M3, layout, dst)
        torch.cuda.synchronize()
        wq, ws = orc.quantize(x, orc.ROW if orientation == ROW else orc.COL)
        want = orc.dequantize(wq, ws, orc.ROW if orientation == ROW else orc.COL, orc.E4M3, name)
        if name == "f32":
            assert np.array_equal(dst.cpu().numpy().view(np.uint32), want.view(np.uint32))
        else:
            assert np.array_equal(dst.view(torch.int16).cpu().numpy().view(np.uint16), want)


def test_quantize_host_variant():
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = 256, 384
    x = synth.f32_to_bf16_bits(synth.gaussian((rows, cols), 3))
    src = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory()
    ws = torch.empty(B.mxfp8_quantize_host_ws_bytes(B.BF16, rows, cols, B.BOTH), dtype=torch.uint8, device="cuda")
    host = [torch.empty(n, dtype=torch.uint8).pin_memory() for n in (
        rows * cols, B.mxfp8_scale_bytes(rows, cols, B.ROW, B.SF_LINEAR),
        rows * cols, B.mxfp8_scale_bytes(rows, cols, B.COL, B.SF_LINEAR))]
    B.mxfp8_quantize_host(src, B.BOTH, B.RULE_PAPER, B.E4M3, host[0], host[1], host[2], host[3], B.SF_LINEAR, ws)
    xf = orc.bf16_bits_to_f32(x)
    wq, wsr = orc.quantize(xf, orc.ROW)
    assert np.array_equal(host[0].numpy().reshape(rows, cols), wq) and np.array_equal(host[1].numpy().reshape(rows, -1), wsr)
    wq, wsc = orc.quantize(xf, orc.COL)
    assert np.array_equal(host[2].numpy().reshape(rows, cols), wq) and np.array_equal(host[3].numpy().reshape(-1, cols), wsc)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("orientation", [ROW, COL, BOTH])
def test_quantize_multi_equals_oracle_per_tensor(dtype, orientation):
    # several tensors of different shapes (ragged tiles, a single-tile tensor) in one launch
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import Guarded, logical_scales_from_swizzled
    shapes = [(160, 352), (32, 32), (384, 1056), (128, 128), (96, 4096 + 128)]
    hosts = [as_dtype(synth.draw(synth.DISTRIBUTIONS[i % 4], s, 900 + i), dtype) for i, s in enumerate(shapes)]
    srcs = [torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(h).cuda()
            for h in hosts]
    outs, entries = [], []
    for (rows, cols), src in zip(shapes, srcs):
        g = {}
        for o, name in ((ROW, "row"), (COL, "col")):
            if orientation & o:
                g["q_" + name] = Guarded(rows * cols)
                g["s_" + name] = Guarded(B.mxfp8_scale_bytes(rows, cols, o, SWIZZLED))
        outs.append(g)
        v = lambda k: g[k].view if k in g else None
        entries.append((src, v("q_row"), v("s_row"), v("q_col"), v("s_col")))
    items = B.make_quantize_items(entries)
    before = B.mxfp8_launch_count()
    B.mxfp8_quantize_multi(items, B.BF16 if dtype == "bf16" else B.FP32, orientation, B.RULE_PAPER, B.E4M3, SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_launch_count() - before == 1
    assert B.mxfp8_device_status() == 0
    for (rows, cols), h, g in zip(shapes, hosts, outs):
        x = orc.bf16_bits_to_f32(h) if dtype == "bf16" else h
        for o, name in ((orc.ROW, "row"), (orc.COL, "col")):
            if ("q_" + name) not in g:
                continue
            g["q_" + name].check(); g["s_" + name].check()
            wq, ws = orc.quantize(x, o, orc.RULE_PAPER, orc.E4M3)
            assert_q_equal(g["q_" + name].numpy().reshape(rows, cols), wq, orc.E4M3, "%s %s" % ((rows, cols), name))
            mn, nkb = (rows, cols // 32) if name == "row" else (cols, rows // 32)
            logical = logical_scales_from_swizzled(g["s_" + name].numpy(), mn, nkb)
            assert np.array_equal(logical if name == "row" else logical.T, ws), "scales %s %s" % ((rows, cols), name)


def test_quantize_multi_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    q, s, _, _ = B.alloc_quantize_outputs(64, 64, B.ROW, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):                      # more tensors than one launch takes
        B.mxfp8_quantize_multi(B.make_quantize_items([(x, q, s, None, None)] * 9), B.BF16, B.ROW, B.RULE_PAPER, B.E4M3, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):                      # missing output
        B.mxfp8_quantize_multi(B.make_quantize_items([(x, q, None, None, None)]), B.BF16, B.ROW, B.RULE_PAPER, B.E4M3, B.SF_LINEAR)
    y = torch.zeros(64, 40, dtype=torch.bfloat16, device="cuda")
    _, _, qc, sc = B.alloc_quantize_outputs(64, 40, B.COL, B.SF_LINEAR)
    with pytest.raises(B.Mxfp8Error):                      # cols % 16 != 0 has no batched path
        B.mxfp8_quantize_multi(B.make_quantize_items([(y, None, None, qc, sc)]), B.BF16, B.COL, B.RULE_PAPER, B.E4M3, B.SF_LINEAR)


def test_more_than_2_to_31_elements_sampled():
    # 40960 x 53248 = 2.18e9 elements (4.4 GB of BF16): every index computation has to be 64-bit.  The oracle
    # checks 128-row slabs at the start, across the 2^31-element mark, and at the very end, for the conversion
    # in both orientations (swizzled scales), the decode of the row copy and the one-pass round trip.
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import logical_scales_from_swizzled
    rows, cols = 40960, 53248
    assert rows * cols > 2 ** 31
    g = torch.Generator(device="cuda"); g.manual_seed(31)
    src = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, rows, 4096):                     # drawn in pieces: no FP32 temporary of the whole tensor
        src[r0:r0 + 4096] = (torch.randn((4096, cols), generator=g, device="cuda") *
                             torch.exp2(torch.randint(-8, 8, (4096, 1), generator=g, device="cuda").float())).to(torch.bfloat16)
    qr, sr, qc, sc = B.alloc_quantize_outputs(rows, cols, B.BOTH, B.SF_SWIZZLED)
    B.mxfp8_quantize(src, B.BOTH, B.RULE_PAPER, B.E4M3, qr, sr, qc, sc, B.SF_SWIZZLED)
    back = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    B.mxfp8_dequantize(qr, sr, B.ROW, B.E4M3, B.SF_SWIZZLED, back)
    fq = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    B.mxfp8_fake_quantize(src, B.ROW, B.RULE_PAPER, B.E4M3, fq, None)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    mark = (2 ** 31) // cols // 128 * 128               # the slab that contains element 2^31
    s_row_raw, s_col_raw = sr.cpu().numpy(), sc.cpu().numpy()
    for r0 in (0, mark, rows - 128):
        sl = slice(r0, r0 + 128)
        x = orc.bf16_bits_to_f32(src[sl].view(torch.int16).cpu().numpy().view(np.uint16))
        wq, ws = orc.quantize(x, orc.ROW)
        m_idx, k_idx = np.meshgrid(np.arange(r0, r0 + 128), np.arange(cols // 32), indexing="ij")
        atoms_k = (cols // 32 + 3) // 4
        off = ((m_idx // 128) * atoms_k + k_idx // 4) * 512 + (m_idx % 32) * 16 + ((m_idx % 128) // 32) * 4 + k_idx % 4
        assert off[-1, -1] == orc.sf_offset_swizzled(r0 + 127, cols // 32 - 1, cols // 32)
        assert np.array_equal(s_row_raw[off], ws)
        assert_q_equal(qr[sl].cpu().numpy(), wq, orc.E4M3, "row slab %d" % r0)
        want = orc.dequantize(wq, ws, orc.ROW, orc.E4M3, "bf16")
        assert np.array_equal(back[sl].view(torch.int16).cpu().numpy().view(np.uint16), want)
        assert np.array_equal(fq[sl].view(torch.int16).cpu().numpy().view(np.uint16), want)
        wq, ws = orc.quantize(x, orc.COL)                # [4, cols] scales of these four 32-row blocks
        c_idx, b_idx = np.meshgrid(np.arange(cols), np.arange(r0 // 32, r0 // 32 + 4), indexing="ij")
        atoms_kc = (rows // 32 + 3) // 4
        offc = ((c_idx // 128) * atoms_kc + b_idx // 4) * 512 + (c_idx % 32) * 16 + ((c_idx % 128) // 32) * 4 + b_idx % 4
        assert np.array_equal(s_col_raw[offc].T, ws)
        assert_q_equal(qc[sl].cpu().numpy(), wq, orc.E4M3, "col slab %d" % r0)


def test_conversions_on_many_streams_at_once():
    """A conversion of many tiles per CTA hands its tiles out through a counter that belongs to the launch's stream.
    Launches that overlap on different streams must not disturb one another, a second launch on a stream must find
    the counter as the first one left it, and streams beyond the number of counters (64) take the fixed tile order:
    the bytes are those of the oracle in every case."""
    import torch
    from paper_2506_08027_b200 import binding as B
    from helpers import logical_scales_from_swizzled
    S = B.SF_SWIZZLED
    thr = os.cpu_count() or 1
    shapes = [(4096, 8192), (2048 + 32, 16384 + 128)]        # 2048 and 2193 tiles of 128 x 128: more than 4 per CTA
    srcs, wants = [], []
    for k, shape in enumerate(shapes):
        bits = synth.f32_to_bf16_bits(synth.gaussian(shape, 400 + k))
        srcs.append(torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16))
        x = orc.bf16_bits_to_f32(bits)
        wants.append((orc.quantize_threads(x, orc.ROW, orc.RULE_PAPER, orc.E4M3, thr),
                      orc.quantize_threads(x, orc.COL, orc.RULE_PAPER, orc.E4M3, thr)))
    streams = [torch.cuda.Stream() for _ in range(70)]
    outs = [[B.alloc_quantize_outputs(*shapes[k % 2], B.BOTH, S) for k in range(len(streams))] for _ in range(2)]
    torch.cuda.synchronize()
    for rep in range(2):                                   # the second round reuses every stream's counter
        for k, st in enumerate(streams):
            with torch.cuda.stream(st):
                B.mxfp8_quantize(srcs[k % 2], B.BOTH, B.RULE_PAPER, B.E4M3, *outs[rep][k], S)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for rep in range(2):
        for k in range(len(streams)):
            (wq_r, ws_r), (wq_c, ws_c) = wants[k % 2]
            rows, cols = shapes[k % 2]
            q_row, s_row, q_col, s_col = outs[rep][k]
            assert np.array_equal(q_row.cpu().numpy(), wq_r), "row bytes, stream %d" % k
            assert np.array_equal(q_col.cpu().numpy(), wq_c), "column bytes, stream %d" % k
            if k < 2 or k >= 68:
                got_r = logical_scales_from_swizzled(s_row.cpu().numpy(), rows, cols // 32)
                got_c = logical_scales_from_swizzled(s_col.cpu().numpy(), cols, rows // 32)
                assert np.array_equal(got_r, ws_r) and np.array_equal(got_c.T, ws_c), "scale bytes, stream %d" % k


@pytest.mark.parametrize("dtype,elem,rule", [("bf16", orc.E5M2, orc.RULE_OCP), ("fp32", orc.E4M3, orc.RULE_PAPER)])
def test_large_ragged_tensor_with_tiles_handed_out_by_the_counter(dtype, elem, rule):
    """More than four tiles per CTA (the stream's tile counter is in use), the last tile of every row and the last
    row of tiles ragged, linear scale layout (the per-row / per-column store path): bytes equal to the oracle's."""
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = 4096 + 32, (8192 + 32 if dtype == "bf16" else 4096 + 32)      # 33 x 65 tiles, the last of each ragged
    thr = os.cpu_count() or 1
    x32 = synth.gaussian((rows, cols), 77)
    src_np = as_dtype(x32, dtype)
    x = orc.bf16_bits_to_f32(src_np) if dtype == "bf16" else src_np
    src = (torch.from_numpy(src_np.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(src_np).cuda())
    q_row, s_row, _, _ = B.alloc_quantize_outputs(rows, cols, B.ROW, B.SF_LINEAR)
    B.mxfp8_quantize(src, B.ROW, rule, elem, q_row, s_row, None, None, B.SF_LINEAR)
    _, _, q_col, s_col = B.alloc_quantize_outputs(rows, cols, B.COL, B.SF_LINEAR)
    B.mxfp8_quantize(src, B.COL, rule, elem, None, None, q_col, s_col, B.SF_LINEAR)
    assert B.mxfp8_device_status() == 0
    wq, ws = orc.quantize_threads(x, orc.ROW, rule, elem, thr)
    assert_q_equal(q_row.cpu().numpy(), wq, elem, "row")
    assert np.array_equal(s_row.cpu().numpy().reshape(rows, cols // 32), ws)
    wq, ws = orc.quantize_threads(x, orc.COL, rule, elem, thr)
    assert_q_equal(q_col.cpu().numpy(), wq, elem, "col")
    assert np.array_equal(s_col.cpu().numpy().reshape(rows // 32, cols), ws)


def test_conversion_captured_in_a_graph_equals_the_eager_one():
    """A launch that is being captured cannot own a stream's tile counter and takes the fixed tile order: the replayed
    graph must give the bytes of the eager call (which, at this size, uses the counter)."""
    import torch
    from paper_2506_08027_b200 import binding as B
    S = B.SF_SWIZZLED
    rows, cols = 4096, 8192
    bits = synth.f32_to_bf16_bits(synth.gaussian((rows, cols), 91))
    src = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    eager = B.alloc_quantize_outputs(rows, cols, B.BOTH, S)
    graph = B.alloc_quantize_outputs(rows, cols, B.BOTH, S)
    B.mxfp8_quantize(src, B.BOTH, B.RULE_PAPER, B.E4M3, *eager, S)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        B.mxfp8_quantize(src, B.BOTH, B.RULE_PAPER, B.E4M3, *graph, S)
    for t in graph:
        t.zero_()
    g.replay(); g.replay()
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for a, b in zip(eager, graph):
        assert torch.equal(a, b)
    wq, _ = orc.quantize_threads(orc.bf16_bits_to_f32(bits), orc.ROW, orc.RULE_PAPER, orc.E4M3, os.cpu_count() or 1)
    assert np.array_equal(eager[0].cpu().numpy(), wq)
