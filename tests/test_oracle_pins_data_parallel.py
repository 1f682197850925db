"""Pins for the oracle's data-parallel step: what the sharded arithmetic must reduce to.

The paper fixes the single-device arithmetic (Sec. 3.2, Sec. 3.3); the sharded step is pinned to it: with the
blocks never crossing a shard, gathering the shards' conversions IS the conversion of the whole weight, and the
sum of the ranks' partial WGRAD products IS the product over all tokens.  A plausible mistake (a shard in the
wrong place, a scale array joined along the wrong axis, a partial product dropped or doubled, dX built from the
row-blocked weight) breaks one of these."""
import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth


def _inputs(world, Tr, H, F, seed):
    xs = [orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.gaussian((Tr, H), seed + 10 * r))) for r in range(world)]
    dys = [orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.output_gradient((Tr, F), seed + 10 * r + 1))) for r in range(world)]
    w = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(0.02 * synth.gaussian((F, H), seed + 5)))
    Fr = F // world
    return xs, [w[r * Fr:(r + 1) * Fr] for r in range(world)], dys, w


def _chain(x, w, dy, rule):
    q = {n: {o: orc.quantize(t, o, rule, orc.E4M3) for o in (orc.ROW, orc.COL)} for n, t in (("x", x), ("w", w), ("dy", dy))}
    R, C = orc.ROW, orc.COL
    y, _ = orc.gemm_f64(q["x"][R][0], q["x"][R][1], q["w"][R][0], q["w"][R][1], "k", "k")
    dx, _ = orc.gemm_f64(q["dy"][R][0], q["dy"][R][1], q["w"][C][0], q["w"][C][1], "k", "mn")
    dw, _ = orc.gemm_f64(q["dy"][C][0], q["dy"][C][1], q["x"][C][0], q["x"][C][1], "mn", "mn")
    return y, dx, dw


@pytest.mark.parametrize("rule", [orc.RULE_PAPER, orc.RULE_OCP])
def test_gathered_shard_conversions_are_the_conversion_of_the_whole_weight(rule):
    _, shards, _, w = _inputs(4, 32, 96, 256, 3)
    for o in (orc.ROW, orc.COL):
        q_full, s_full = orc.quantize(w, o, rule)
        parts = [orc.quantize(sh, o, rule) for sh in shards]
        assert np.array_equal(np.concatenate([q for q, _ in parts]), q_full)
        assert np.array_equal(np.concatenate([sc for _, sc in parts]), s_full)   # ROW: [F, H/32]; COL: [F/32, H]: both stack by rows


@pytest.mark.parametrize("world", [1, 2, 4])
def test_sharded_step_equals_the_single_device_step_on_all_tokens(world):
    Tr, H, F = 64, 96, 128 * world if world > 1 else 128
    xs, shards, dys, w = _inputs(world, Tr, H, F, 11)
    ys, dxs, dws, sabs = orc.data_parallel_linear_f64(xs, shards, dys)
    y, dx, dw = _chain(np.concatenate(xs), w, np.concatenate(dys), orc.RULE_PAPER)
    # per-rank products involve the rank's own rows only: the rows of the whole product (up to the order of binary64 sums)
    assert np.abs(np.concatenate(ys) - y).max() <= 1e-13 * np.concatenate(sabs[0]).max()
    assert np.abs(np.concatenate(dxs) - dx).max() <= 1e-13 * np.concatenate(sabs[1]).max()
    # dW: a sum over ranks of binary64 partial sums against one binary64 sum over all tokens
    got = np.concatenate(dws)
    assert got.shape == dw.shape
    assert np.abs(got - dw).max() <= 1e-13 * np.concatenate(sabs[2]).max()
    for r in range(world):
        assert dws[r].shape == shards[r].shape


def test_sharded_wgrad_counts_every_rank_once():
    """A rank whose output gradient is zero adds nothing; doubling one rank's gradient doubles only its part."""
    xs, shards, dys, _ = _inputs(2, 32, 64, 256, 23)
    _, _, base, _ = orc.data_parallel_linear_f64(xs, shards, dys)
    _, _, only0, _ = orc.data_parallel_linear_f64(xs, shards, [dys[0], np.zeros_like(dys[1])])
    _, _, only1, _ = orc.data_parallel_linear_f64(xs, shards, [np.zeros_like(dys[0]), dys[1]])
    _, _, twice1, _ = orc.data_parallel_linear_f64(xs, shards, [dys[0], 2.0 * dys[1]])   # a power of two: scales move, codes stay
    for r in range(2):
        assert np.allclose(only0[r] + only1[r], base[r], rtol=1e-13, atol=0)
        assert np.allclose(only0[r] + 2.0 * only1[r], twice1[r], rtol=1e-13, atol=0)


def test_concat_of_swizzled_scales_is_the_swizzle_of_the_concatenation():
    rng = np.random.default_rng(5)
    mn, nkb_part, parts_n = 200, 8, 3
    logical = [rng.integers(0, 255, size=(mn, nkb_part), dtype=np.uint8) for _ in range(parts_n)]
    got = orc.concat_swizzled_scales_k([orc.swizzle_scales(p) for p in logical], mn, nkb_part)
    assert np.array_equal(got, orc.swizzle_scales(np.concatenate(logical, axis=1)))
    # column-blocked scales of row shards: linear layout [F_r/32, H] per shard, logical [H, F/32] for the GEMM
    w = rng.standard_normal((256, 64)).astype(np.float32)
    shards = [w[:128], w[128:]]
    s_parts = [orc.swizzle_scales(np.ascontiguousarray(orc.quantize(sh, orc.COL)[1].T)) for sh in shards]
    s_full = orc.swizzle_scales(np.ascontiguousarray(orc.quantize(w, orc.COL)[1].T))
    assert np.array_equal(orc.concat_swizzled_scales_k(s_parts, 64, 4), s_full)
