// Device-side building blocks of the MXFP8 conversion (sm_100a only).
//
// Paper passages implemented here: UE8M0 scale from the block amax (Algorithm 1 and the
// bit-space order of App. A.1, plus the OCP v1.0 rule of Sec. 3.3), and Quantize_to_fp8
// (Sec. 3.3, App. A.2) through the hardware's saturating round-to-nearest-even converts.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxfp8.h"

namespace mxfp8 {

// Per element type (Table 1): exponent of the largest normal, and the FP32 mantissa field of the
// largest normal (448 = 1.75*2^8, 57344 = 1.75*2^15, 7.5 = 1.875*2^2, 28 = 1.75*2^4, 6 = 1.5*2^2).
// paper_offset, added to the bit pattern of amax, carries into the exponent field exactly when the
// mantissa of amax exceeds that of the largest normal, i.e. when amax/destmax rounds up a binade.
template <int ELEM> struct ElemTraits;
template <> struct ElemTraits<MXFP8_E4M3> { static constexpr int emax = 8;  static constexpr uint32_t max_mant = 0x600000u; };
template <> struct ElemTraits<MXFP8_E5M2> { static constexpr int emax = 15; static constexpr uint32_t max_mant = 0x600000u; };
template <> struct ElemTraits<MXFP8_E2M3> { static constexpr int emax = 2;  static constexpr uint32_t max_mant = 0x700000u; };
template <> struct ElemTraits<MXFP8_E3M2> { static constexpr int emax = 4;  static constexpr uint32_t max_mant = 0x600000u; };
template <> struct ElemTraits<MXFP8_E2M1> { static constexpr int emax = 2;  static constexpr uint32_t max_mant = 0x400000u; };
template <int ELEM> __host__ __device__ constexpr uint32_t paper_offset() { return 0x7FFFFFu - ElemTraits<ELEM>::max_mant; }

// UE8M0 byte from the FP32 bit pattern of a finite, non-negative amax.
// destmax = 1.m_max * 2^emax (m_max = ElemTraits::max_mant), so with E the biased
// exponent field of amax:   amax/destmax = (1.m / 1.m_max) * 2^(E - 127 - emax).
//   paper rule: round that ratio up to a power of two -> exponent E-127-emax, plus one when
//               1.m > 1.m_max; clamp below at -127 (byte 0).  FP32-subnormal amax (E == 0) is
//               far below destmax * 2^-127, so its byte is 0.
//   ocp rule  : floor(log2 amax) - emax = E - 127 - emax, clamped (subnormal amax -> byte 0).
// The upper clamp never binds: the largest byte an FP32 amax can give is 247.
template <int ELEM>
__device__ __forceinline__ uint32_t scale_byte_from_amax_bits(uint32_t amax_bits, int rule)
{
    const int e_field = (int)(amax_bits >> 23);
    const int up = (rule == MXFP8_RULE_PAPER) && ((amax_bits & 0x7FFFFFu) > ElemTraits<ELEM>::max_mant);
    int b = e_field - ElemTraits<ELEM>::emax + up;
    b = (e_field == 0) ? 0 : b;
    return (uint32_t)max(b, 0);
}

// 2^(127-b) = 1/X as an FP32 value; b <= 247 so the exponent field stays >= 7 (normal).
__device__ __forceinline__ float inv_scale_from_byte(uint32_t b)
{
    return __uint_as_float((254u - b) << 23);
}

// Two FP32 values -> two element codes, round-to-nearest-even, saturating to +-destmax,
// NaN -> NaN where the format has one.  Result: one code per byte (6- and 4-bit codes in the low
// bits of their byte), `lo` in bits 0-7, `hi` in bits 8-15.
template <int ELEM>
__device__ __forceinline__ uint32_t cvt_fp8x2(float lo, float hi)
{
    uint16_t r;
    if constexpr (ELEM == MXFP8_E4M3)
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else if constexpr (ELEM == MXFP8_E5M2)
        asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else if constexpr (ELEM == MXFP8_E2M3)
        asm("cvt.rn.satfinite.e2m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else if constexpr (ELEM == MXFP8_E3M2)
        asm("cvt.rn.satfinite.e3m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else {
        // the 4-bit convert packs both codes into one byte (first operand in the high nibble)
        asm("{\n\t.reg .b8 t;\n\tcvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\tcvt.u16.u8 %0, t;\n\t}" : "=h"(r) : "f"(hi), "f"(lo));
        r = (uint16_t)((r & 0x0Fu) | ((r & 0xF0u) << 4));
    }
    return (uint32_t)r;
}

template <int ELEM>
__device__ __forceinline__ uint32_t cvt_fp8x4(float a, float b, float c, float d)
{
    return cvt_fp8x2<ELEM>(a, b) | (cvt_fp8x2<ELEM>(c, d) << 16);
}

// Two element codes (one per byte, bits 0-15) -> two FP32 values (exact: every element value is an FP16 value).
template <int ELEM>
__device__ __forceinline__ float2 fp8x2_to_float2(uint32_t two_codes)
{
    uint32_t h2;
    uint16_t in = (uint16_t)two_codes;
    if constexpr (ELEM == MXFP8_E4M3)
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(in));
    else if constexpr (ELEM == MXFP8_E5M2)
        asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(in));
    else if constexpr (ELEM == MXFP8_E2M3) {
        in &= 0x3F3Fu;                       // bits above a 6-bit code are ignored
        asm("cvt.rn.f16x2.e2m3x2 %0, %1;" : "=r"(h2) : "h"(in));
    } else if constexpr (ELEM == MXFP8_E3M2) {
        in &= 0x3F3Fu;
        asm("cvt.rn.f16x2.e3m2x2 %0, %1;" : "=r"(h2) : "h"(in));
    } else {
        in = (uint16_t)((in & 0x0Fu) | ((in >> 4) & 0xF0u));      // two nibbles in one byte
        asm("{\n\t.reg .b8 t;\n\tcvt.u8.u16 t, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, t;\n\t}" : "=r"(h2) : "h"(in));
    }
    __half2 h = *reinterpret_cast<__half2*>(&h2);
    return __half22float2(h);
}

// Byte offset of scale (mn, kb) in the 128x4 atom layout (see mxfp8.h).
__host__ __device__ __forceinline__ int64_t sf_swizzled_offset(int64_t mn, int64_t kb, int64_t n_kblocks)
{
    const int64_t atoms_k = (n_kblocks + 3) >> 2;
    return ((mn >> 7) * atoms_k + (kb >> 2)) * 512 + (mn & 31) * 16 + ((mn >> 5) & 3) * 4 + (kb & 3);
}

}  // namespace mxfp8
