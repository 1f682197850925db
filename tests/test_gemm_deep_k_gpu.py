"""Parity of mxfp8_gemm with the FP64 oracle at the deepest reductions and the largest products.

Sec. 2 / App. A.3 define the product as block dot products, each scaled by its two blocks' scales and
accumulated in FP32.  How the tensor core orders and aligns that accumulation is not specified, so the
acceptance bound is a tolerance: |D - D64| <= 2^-16 * sum_k |a_k b_k| per element and a relative
Frobenius error <= 1e-5.  An FP32 running sum loses about sqrt(K) * 2^-24 relative to the magnitude
sum, which reaches 2^-16 at K = 65536: these cases measure how much of the bound the kernel uses there.

Shapes: the skinny WGRAD of the GEMM sweep (4096 x 4096 x 65536, both operands token-major), 16384^3,
and one product of the 8B decoder block per (majors, K) class.  Sources are drawn on the device with a
seeded generator; the oracle converts the same source bytes on the host (the whole B operand, sampled
rows of A: first, last, tile edges, random), and its bytes for B must equal the device's.
"""
import json
import os

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth
from helpers import check_gemm_tolerance

pytestmark = pytest.mark.gpu


def _host_f32(t):
    import torch
    return orc.bf16_bits_to_f32(t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))


def _sampled_rows(M, seed, n_random=37):
    rng = np.random.default_rng(seed)
    edges = [0, 1, 127, 128, 255, 256, M - 257, M - 256, M - 129, M - 128, M - 1]
    return np.unique(np.concatenate([edges, rng.integers(0, M, n_random)]))


def _report(entry):
    path = os.environ.get("MXFP8_PARITY_REPORT")
    if path:
        with open(path, "a") as fh:
            fh.write(json.dumps(entry) + "\n")


CASES = [
    # name, M, N, K, A major, B major, kind of A, kind of B
    ("skinny wgrad 4096x4096x65536", 4096, 4096, 65536, "mn", "mn", "output_gradient", "activation"),
    ("square 16384^3", 16384, 16384, 16384, "k", "k", "gaussian", "gaussian"),
    ("ffn_up fprop 16384x28672x4096", 16384, 28672, 4096, "k", "k", "activation", "weight"),
    ("ffn_down fprop 16384x4096x14336", 16384, 4096, 14336, "k", "k", "activation", "weight"),
    ("ffn_up dgrad 16384x4096x28672", 16384, 4096, 28672, "k", "mn", "output_gradient", "weight"),
    ("qkv wgrad 6144x4096x16384", 6144, 4096, 16384, "mn", "mn", "output_gradient", "activation"),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0].split(" ")[0] + "_" + c[0].split(" ")[1] for c in CASES])
def test_deep_and_large_products_against_the_fp64_oracle(case):
    import torch
    from paper_2506_08027_b200 import binding as B
    name, M, N, K, am, bm, kind_a, kind_b = case
    thr = os.cpu_count() or 1
    S = B.SF_SWIZZLED
    seed = 9000 + 13 * len(name) + K % 997

    def device_operand(mn, major, kind, sd):
        shape = (mn, K) if major == "k" else (K, mn)
        src = synth.device_tensor(kind, shape, sd)
        o = B.ROW if major == "k" else B.COL
        outs = B.alloc_quantize_outputs(shape[0], shape[1], o, S)
        B.mxfp8_quantize(src, o, B.RULE_PAPER, B.E4M3, *outs, S)
        return src, (outs[0], outs[1]) if major == "k" else (outs[2], outs[3])

    a_src, (Aq, As) = device_operand(M, am, kind_a, seed)
    b_src, (Bq, Bs) = device_operand(N, bm, kind_b, seed + 1)
    D = torch.empty((M, N), dtype=torch.float32, device="cuda")
    B.mxfp8_gemm(Aq, As, Bq, Bs, M, N, K, B.MN_MAJOR if am == "mn" else B.K_MAJOR,
                 B.MN_MAJOR if bm == "mn" else B.K_MAJOR, B.E4M3, B.E4M3, D)
    assert B.mxfp8_device_status() == 0

    # the oracle's own conversion of the same sources: all of B, the sampled rows of A
    rows = _sampled_rows(M, seed)
    rows_d = torch.from_numpy(rows).cuda()
    bq, bs = orc.quantize_threads(_host_f32(b_src), orc.ROW if bm == "k" else orc.COL, orc.RULE_PAPER, orc.E4M3, thr)
    assert np.array_equal(Bq.cpu().numpy(), bq), "device and oracle conversions of B differ"
    del b_src
    if am == "k":
        a_sub = _host_f32(a_src[rows_d])
        aq, a_s = orc.quantize(a_sub, orc.ROW)
        assert np.array_equal(Aq[rows_d].cpu().numpy(), aq)
    else:
        a_sub = _host_f32(a_src[:, rows_d])
        aq, a_s = orc.quantize_threads(a_sub, orc.COL, orc.RULE_PAPER, orc.E4M3, thr)
        assert np.array_equal(Aq[:, rows_d].cpu().numpy(), aq)
    del a_src
    d64, sabs = orc.gemm_f64(aq, a_s, bq, bs, am, bm)
    got = D[rows_d].cpu().numpy()
    # the two figures first (kept in the report whatever the verdict), then the acceptance bounds
    err = np.abs(got.astype(np.float64) - d64)
    worst = float((err / (2.0 ** -16 * sabs + 2.0 ** -126)).max())
    fro = float(np.sqrt((err ** 2).sum()) / np.sqrt((d64 ** 2).sum()))
    toward_zero = float((np.abs(got.astype(np.float64)) < np.abs(d64)).mean())   # 0.5 for unbiased rounding
    _report({"case": name, "M": M, "N": N, "K": K, "majors": am + " x " + bm, "rows_checked": int(rows.size),
             "worst_err_over_bound": worst, "rel_frobenius": fro, "share_smaller_in_magnitude": toward_zero})
    print("%s: worst err / (2^-16 sum|ab|) = %.4f, relative Frobenius error %.3g, |D| < |D64| on %.1f %% of the elements"
          % (name, worst, fro, 100 * toward_zero))
    check_gemm_tolerance(got, d64, sabs, name)
