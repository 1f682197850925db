"""CPU oracle for the MXFP8 conversion and block-scaled GEMM -- TEST INFRASTRUCTURE.

Nothing in the product imports this package.  Only the tests, the smoke check and
the benchmark's CPU-baseline / reference legs may use it.  It is written from the
paper ("Recipes for Pre-training LLMs with MXFP8": Sec. 2, Sec. 3.2, Sec. 3.3,
Algorithm 1, App. A.1, App. A.2, Table 1) and shares no code with the CUDA path.
"""
from .mxfp8_oracle import (  # noqa: F401
    E4M3, E5M2, E2M3, E3M2, E2M1, RULE_PAPER, RULE_OCP, ROW, COL,
    build_oracle, fp8_decode, fp8_encode, scale_byte, quantize, dequantize_f64,
    dequantize, bf16_bits_to_f32, sf_offset_swizzled,
    swizzle_scales, gemm_f64, quantize_threads, grouped_gemm_f64, code_bits, pack_codes16, unpack_codes16,
    ACT_NONE, ACT_RELU, ACT_RELU2, ACT_SILU, ACT_GELU_TANH, activation, rmsnorm, glu, layernorm, activation_grad,
    concat_swizzled_scales_k, data_parallel_linear_f64,
)
