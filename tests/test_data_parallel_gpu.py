"""The two exchange kernels of the data-parallel step, on one GPU: joining swizzled scales of gathered weight
shards, and the WGRAD product that adds its result into per-owner buffers (ranks emulated as consecutive
launches that write into owner buffers on the same device; no launch waits for another)."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import check_gemm_tolerance, swizzle_np

pytestmark = pytest.mark.gpu


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("mn,k_part,parts", [(128, 128, 2), (200, 256, 3), (2048, 1024, 8), (64, 128, 1)])
def test_sf_concat_k_matches_oracle(mn, k_part, parts):
    import torch
    from paper_2506_08027_b200 import binding as B
    rng = np.random.default_rng(mn + parts)
    logical = [rng.integers(0, 255, size=(mn, k_part // 32), dtype=np.uint8) for _ in range(parts)]
    swz = [swizzle_np(p) for p in logical]
    want = swizzle_np(np.concatenate(logical, axis=1))
    if mn * k_part * parts <= 200 * 256 * 3:
        assert np.array_equal(orc.concat_swizzled_scales_k(swz, mn, k_part // 32), want)   # the fast form used for the large cases
    src = _dev(np.concatenate(swz))
    dst = torch.full((want.size + 64,), 0xEE, dtype=torch.uint8, device="cuda")
    B.mxfp8_sf_concat_k(src, parts, mn, k_part, dst[:want.size])
    torch.cuda.synchronize()
    got = dst.cpu().numpy()
    assert np.array_equal(got[:want.size], want)
    assert (got[want.size:] == 0xEE).all()


@pytest.mark.parametrize("world", [2, 4])
def test_shard_conversions_written_at_their_row_offset_assemble_the_whole_weight(world):
    """Element bytes of both orientations and the row-blocked scales land in place; the column-blocked scales go
    through mxfp8_sf_concat_k.  The result must be, byte for byte, the conversion of the whole weight."""
    import torch
    from paper_2506_08027_b200 import binding as B
    F, H = 256 * world, 384
    Fr = F // world
    wb = synth.f32_to_bf16_bits(0.02 * synth.gaussian((F, H), 91))
    w = torch.from_numpy(wb.view(np.int16)).cuda().view(torch.bfloat16)
    u8 = dict(dtype=torch.uint8, device="cuda")
    full = dict(q_row=torch.empty(F, H, **u8), q_col=torch.empty(F, H, **u8),
                s_row=torch.empty(B.mxfp8_scale_bytes(F, H, B.ROW, B.SF_SWIZZLED), **u8),
                s_col=torch.empty(B.mxfp8_scale_bytes(F, H, B.COL, B.SF_SWIZZLED), **u8))
    B.mxfp8_quantize(w, B.BOTH, B.RULE_PAPER, B.E4M3, full["q_row"], full["s_row"], full["q_col"], full["s_col"], B.SF_SWIZZLED)
    got = {k: torch.full_like(v, 0xEE) for k, v in full.items()}
    srow_part = B.mxfp8_scale_bytes(Fr, H, B.ROW, B.SF_SWIZZLED)
    scol_part = B.mxfp8_scale_bytes(Fr, H, B.COL, B.SF_SWIZZLED)
    parts = torch.empty(world * scol_part, **u8)
    for r in range(world):
        B.mxfp8_quantize(w[r * Fr:(r + 1) * Fr], B.BOTH, B.RULE_PAPER, B.E4M3,
                         got["q_row"][r * Fr:(r + 1) * Fr], got["s_row"][r * srow_part:(r + 1) * srow_part],
                         got["q_col"][r * Fr:(r + 1) * Fr], parts[r * scol_part:(r + 1) * scol_part], B.SF_SWIZZLED)
    B.mxfp8_sf_concat_k(parts, world, H, Fr, got["s_col"])
    torch.cuda.synchronize()
    for k in full:
        assert torch.equal(got[k], full[k]), k


def _wgrad_operands(T, H, F, seed):
    """dY [T, F] and X [T, H] converted with blocks running down the token axis (WGRAD's reduction axis)."""
    x = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.gaussian((T, H), seed)))
    dy = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.output_gradient((T, F), seed + 1)))
    return orc.quantize(dy, orc.COL), orc.quantize(x, orc.COL)


def _scatter(dyq, xq, owners, first_owner):
    from paper_2506_08027_b200 import binding as B
    (aq, a_s), (bq, b_s) = dyq, xq
    T, F = aq.shape
    H = bq.shape[1]
    B.mxfp8_gemm_reduce_scatter(_dev(aq), _dev(swizzle_np(np.ascontiguousarray(a_s.T))), _dev(bq), _dev(swizzle_np(np.ascontiguousarray(b_s.T))),
                                F, H, T, B.MN_MAJOR, B.MN_MAJOR, B.E4M3, B.E4M3, B.make_owner_pointers(owners), first_owner)
    assert B.mxfp8_device_status() == 0


@pytest.mark.parametrize("shape", [(128, 128, 128), (256, 384, 512), (384, 208, 1024)])
def test_reduce_scatter_with_one_owner_is_the_plain_product(shape):
    import torch
    from helpers import gpu_gemm
    T, H, F = shape
    dyq, xq = _wgrad_operands(T, H, F, 7 + T)
    want = gpu_gemm(dyq[0], dyq[1], xq[0], xq[1], "mn", "mn")
    out = torch.zeros(F, H, dtype=torch.float32, device="cuda")
    _scatter(dyq, xq, [out], 0)
    assert np.array_equal(out.cpu().numpy(), want)          # 0 + x = x
    _scatter(dyq, xq, [out], 0)
    assert np.array_equal(out.cpu().numpy(), want + want)    # the call adds: x + x is exact


@pytest.mark.parametrize("world,Tr,H,F", [(2, 128, 256, 512), (4, 256, 320, 1024), (8, 128, 128, 1024), (3, 128, 256, 384)])
def test_reduce_scatter_over_emulated_ranks(world, Tr, H, F):
    """Every 'rank' holds its own tokens and adds its partial product into all owners' row ranges."""
    import torch
    from helpers import gpu_gemm
    Fr = F // world
    owners = [torch.zeros(Fr, H, dtype=torch.float32, device="cuda") for _ in range(world)]
    xs, dys, partials = [], [], []
    for r in range(world):
        dyq, xq = _wgrad_operands(Tr, H, F, 100 * world + 10 * r)
        _scatter(dyq, xq, owners, r)                         # rank r starts at its own rows
        partials.append(gpu_gemm(dyq[0], dyq[1], xq[0], xq[1], "mn", "mn"))
        dys.append(orc.dequantize_f64(dyq[0], dyq[1], orc.COL)); xs.append(orc.dequantize_f64(xq[0], xq[1], orc.COL))
    got = np.concatenate([o.cpu().numpy() for o in owners])
    # launches follow one another on one stream here, so the additions happened in rank order, in FP32
    acc = np.zeros((F, H), dtype=np.float32)
    for part in partials:
        acc = acc + part
    assert np.array_equal(got, acc)
    # and against the definition: the product over all ranks' tokens
    d64 = sum(dy.T @ x for dy, x in zip(dys, xs))
    sabs = sum(np.abs(dy).T @ np.abs(x) for dy, x in zip(dys, xs))
    check_gemm_tolerance(got, d64, world * sabs, "sum of %d partial products" % world)


@pytest.mark.parametrize("tile", ["256p", "192p", "128"])
def test_reduce_scatter_with_every_tile_shape_built_for_it(tile, monkeypatch):
    """The three tile shapes of this mode forced in turn (the library reads MXFP8_GEMM_TILE at every launch): owners' row
    ranges that start inside a 256-row pair tile, a ragged last column tile."""
    import torch
    from helpers import gpu_gemm
    monkeypatch.setenv("MXFP8_GEMM_TILE", tile)
    world, Tr, H, F = 3, 256, 336, 384                     # 128 rows per owner: every pair tile spans two owners
    owners = [torch.zeros(F // world, H, dtype=torch.float32, device="cuda") for _ in range(world)]
    acc = np.zeros((F, H), dtype=np.float32)
    for r in range(world):
        dyq, xq = _wgrad_operands(Tr, H, F, 500 + 10 * r)
        _scatter(dyq, xq, owners, r)
        acc = acc + gpu_gemm(dyq[0], dyq[1], xq[0], xq[1], "mn", "mn")
    assert np.array_equal(np.concatenate([o.cpu().numpy() for o in owners]), acc)


def test_reduce_scatter_argument_errors():
    import torch
    from paper_2506_08027_b200 import binding as B
    u8 = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    out = torch.zeros(128, 128, dtype=torch.float32, device="cuda")
    def call(M=256, N=128, K=128, owners=(out, out), first=0):
        return B.lib().mxfp8_gemm_reduce_scatter(u8.data_ptr(), u8.data_ptr(), u8.data_ptr(), u8.data_ptr(), M, N, K, B.MN_MAJOR, B.MN_MAJOR,
                                                 B.E4M3, B.E4M3, B.make_owner_pointers(list(owners)), len(owners), first, None)
    assert call(M=384) == B.ERR_UNSUPPORTED          # rows per owner must be whole 128-row tiles
    assert call(first=2) == B.ERR_SHAPE
    assert call(owners=[out] * 9, M=9 * 128) == B.ERR_SHAPE
    assert call(K=100) == B.ERR_SHAPE
    assert call(owners=[out, 0]) == B.ERR_NULL
    assert call(owners=[out, out.data_ptr() + 4]) == B.ERR_ALIGN
    assert B.lib().mxfp8_sf_concat_k(u8.data_ptr(), 2, 128, 100, u8.data_ptr(), None) == B.ERR_SHAPE
    assert B.lib().mxfp8_sf_concat_k(None, 2, 128, 128, u8.data_ptr(), None) == B.ERR_NULL
