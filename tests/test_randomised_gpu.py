"""Seeded random sweeps over shapes, element formats, operand majors, scale rules and layouts: combinations the
hand-picked cases do not enumerate.  Quantization bit for bit against the oracle, the GEMM inside its bounds."""
import numpy as np
import pytest

import oracle as orc
from helpers import check_against_oracle, check_gemm_tolerance, gpu_gemm

pytestmark = pytest.mark.gpu
ELEMS = [orc.E4M3, orc.E5M2, orc.E2M3, orc.E3M2, orc.E2M1]


def _packed(q, elem):
    return orc.pack_codes16(q, elem) if orc.code_bits(elem) < 8 else q


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_gemm_random_shapes_formats_and_majors(seed):
    rng = np.random.default_rng(1000 + seed)
    for it in range(12):
        a_major, b_major = rng.choice(["k", "mn"]), rng.choice(["k", "mn"])
        ae, be = int(rng.choice(ELEMS)), int(rng.choice(ELEMS))
        K = int(rng.integers(1, 40)) * 32
        M = int(rng.integers(1, 45)) * 16
        N = int(rng.integers(1, 45)) * 16
        if a_major == "k" and rng.random() < 0.5:
            M = int(rng.integers(1, 700))                 # K-major rows need no alignment
        if b_major == "k" and rng.random() < 0.5:
            N = int(rng.integers(1, 175)) * 4             # FP32 output rows of 16 bytes
        A = (rng.standard_normal((M, K)) * np.exp(rng.normal(0, 2, (M, 1)))).astype(np.float32)
        Bm = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
        aq, a_s = orc.quantize(A, orc.ROW, orc.RULE_PAPER, ae) if a_major == "k" else orc.quantize(np.ascontiguousarray(A.T), orc.COL, orc.RULE_PAPER, ae)
        bq, b_s = orc.quantize(Bm, orc.ROW, orc.RULE_PAPER, be) if b_major == "k" else orc.quantize(np.ascontiguousarray(Bm.T), orc.COL, orc.RULE_PAPER, be)
        d64, sabs = orc.gemm_f64(aq, a_s, bq, b_s, a_major, b_major, ae, be)
        got = gpu_gemm(_packed(aq, ae), a_s, _packed(bq, be), b_s, a_major, b_major, ae, be)
        check_gemm_tolerance(got, d64, sabs, "case %d: M %d N %d K %d %s/%s elems %d/%d" % (it, M, N, K, a_major, b_major, ae, be))


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_quantize_random_shapes_dtypes_rules_and_layouts(seed):
    from paper_2506_08027_b200 import binding as B
    from paper_2506_08027_b200 import synth
    rng = np.random.default_rng(2000 + seed)
    for it in range(14):
        orientation = int(rng.choice([B.ROW, B.COL, B.BOTH]))
        elem = int(rng.choice(ELEMS))
        rule = int(rng.choice([B.RULE_PAPER, B.RULE_OCP]))
        layout = int(rng.choice([B.SF_LINEAR, B.SF_SWIZZLED]))
        dtype = str(rng.choice(["fp32", "bf16"]))
        rows = int(rng.integers(1, 20)) * 32 if orientation & B.COL else int(rng.integers(1, 600))
        cols = int(rng.integers(1, 40)) * 32 if (orientation & B.ROW or orc.code_bits(elem) < 8) else int(rng.integers(1, 300)) * 4
        x = (rng.standard_normal((rows, cols)) * np.exp2(rng.integers(-30, 20, (rows, 1)))).astype(np.float32)
        x[rng.random((rows, cols)) < 0.01] *= 100.0
        if rng.random() < 0.3:                             # a few specials: the careful path of a slab
            idx = rng.integers(0, rows * cols, 5)
            x.reshape(-1)[idx] = rng.choice([np.inf, -np.inf, np.nan, 0.0, -0.0], 5)
        src = synth.f32_to_bf16_bits(x) if dtype == "bf16" else x
        check_against_oracle(src, dtype, orientation, rule, elem, layout,
                             "case %d: %dx%d %s orient %d elem %d rule %d layout %d" % (it, rows, cols, dtype, orientation, elem, rule, layout))
