// Fast path of mxfp8_quantize: TMA in, math, coalesced stores out (Sec. 3.2 / 3.3, Algorithm 1,
// App. A.1-A.2).
//
// The generic kernel in quantize.cu spends most of its issue slots on global address
// arithmetic and predicates.  Here a CTA owns tiles of 128 rows x 256 bytes (128 BF16 or 64 FP32
// columns).  TMA tensor loads bring them into a two-deep shared-memory ring (ragged edges are
// zero-filled by the hardware, the next tile is in flight while the current one is processed),
// the arithmetic reads shared memory at compile-time offsets, and the FP8 bytes go straight to
// global memory: every warp store covers 128 (BF16) or 64 (FP32) contiguous bytes of one row.
//
//   warp w owns rows 32w .. 32w+31 of the tile; lane l owns 8 bytes (4 BF16 / 2 FP32) of every row
//   pass A (column blocks): amax down the 32 rows inside the lane, packed bf16x2 max for BF16
//   pass B (row blocks)   : amax across the lanes of a 32-column block by xor-shuffles; BF16 rows
//                           go through the shuffles two at a time (one in each half of a register)
//   scale: integer form of Algorithm 1 / App. A.1 on the amax bit pattern (see mxfp8_device.cuh); the two BF16 rows of a
//          pair keep sharing one register through it (16-bit lanes).  The bytes wait in shared memory in the order of a
//          swizzled atom and leave once per tile: 16 bytes per lane for a whole BF16 tile, one word per row / column else
//   cast : x * 2^-e in FP32 (exact), cvt.rn.satfinite to the element type (e4m3x2 / e5m2x2, or the
//          6- / 4-bit types, whose codes are then packed 16 to a 16-byte slot across the lanes)
//   One launch takes up to 8 tensors (their tiles form one pool); optional in-place prologues on the
//   tile in shared memory: an activation function or an RMS normalisation ahead of the conversion;
//   optional store mode that writes the decoded values back instead of the codes (round trip).
#pragma once

#include <cuda.h>

#include "mxfp8_device.cuh"
#include "mxfp8_host.h"

namespace mxfp8 {
namespace {

constexpr int T_ROWS = 128;
constexpr int T_BYTES = 256;                 // source bytes per tile row
constexpr int IN_BYTES = T_ROWS * T_BYTES;   // 32 KB
constexpr int QT_THREADS = 128;
constexpr int RING = 2;                      // slots of the input ring
constexpr int QT_CTAS_PER_SM = 3;            // by shared memory (2 x 32 KB + staging) and by registers (168)
// Scale bytes of a tile wait in shared memory in the order of one swizzled 128 x 4 atom (see mxfp8.h): those of row
// (or column) i of the tile start at stage_offset(i), one byte per block, 16 bytes from those of row i + 1.  A whole
// BF16 tile's scales in the swizzled layout are exactly one atom, which then leaves as 32 16-byte stores.
constexpr int STAGE_PITCH = 16;
__device__ __forceinline__ int stage_offset(int i) { return (i & 31) * STAGE_PITCH + (i >> 5) * 4; }
#ifdef MXFP8_TEST_HOOKS
constexpr uint64_t QT_WAIT_LIMIT_NS = 5000000ull;      // test build: the bounded wait gives up after 5 ms
#else
constexpr uint64_t QT_WAIT_LIMIT_NS = 1000000000ull;
#endif

struct QParams {
    int64_t rows, cols;
    int rule, sf_layout;
    int tiles_x, tiles_y;
    uint32_t tiles_x_magic;                  // div_magic(tiles_x)
    uint8_t* q_row;
    uint8_t* q_col;
    uint8_t* s_row;
    uint8_t* s_col;
};

// ACT codes above this offset stand for the derivative of the activation (backward pass: act'(z) * dh)
constexpr int ACT_GRAD = 4;

// Elementwise activation ahead of the conversion (Sec. 3.2 keeps the activation function in high
// precision; its result is what gets converted): evaluated in FP32.  relu(x) = x > 0 ? x : 0 (NaN -> 0).
template <int ACT>
__device__ __forceinline__ float apply_act(float x)
{
    if constexpr (ACT == MXFP8_ACT_RELU) return x > 0.f ? x : 0.f;
    else if constexpr (ACT == MXFP8_ACT_RELU2) return x > 0.f ? x * x : 0.f;
    else if constexpr (ACT == MXFP8_ACT_SILU) return __fdividef(x, 1.f + __expf(-x));
    else if constexpr (ACT == MXFP8_ACT_GELU_TANH) {
        // 0.5 x (1 + tanh(u)) = x / (1 + exp(-2u)), u = sqrt(2/pi) (x + 0.044715 x^3)
        const float u2 = 1.5957691216057308f * (x + 0.044715f * x * x * x);
        return __fdividef(x, 1.f + __expf(-u2));
    } else if constexpr (ACT == ACT_GRAD + MXFP8_ACT_RELU) return x > 0.f ? 1.f : 0.f;
    else if constexpr (ACT == ACT_GRAD + MXFP8_ACT_RELU2) return x > 0.f ? 2.f * x : 0.f;
    else if constexpr (ACT == ACT_GRAD + MXFP8_ACT_SILU) {
        const float sg = __fdividef(1.f, 1.f + __expf(-x));
        return sg * (1.f + x * (1.f - sg));
    } else if constexpr (ACT == ACT_GRAD + MXFP8_ACT_GELU_TANH) {
        // with s = 1 / (1 + exp(-2u)): 0.5 (1 + tanh u) = s and 1 - tanh^2 u = 4 s (1 - s), so
        // gelu'(x) = s + x s (1 - s) * 2 sqrt(2/pi) (1 + 3 * 0.044715 x^2)
        const float u2 = 1.5957691216057308f * (x + 0.044715f * x * x * x);
        const float sg = __fdividef(1.f, 1.f + __expf(-u2));
        return sg + x * sg * (1.f - sg) * (1.5957691216057308f * (1.f + 0.134145f * x * x));
    } else return x;
}

// Applies ACT in place to the 8 bytes per row this lane owns in its 32-row slab, rounding once to the source dtype.
template <int ACT, bool BF>
__device__ __forceinline__ void act_slab(uint8_t* mine)
{
#pragma unroll 8
    for (int j = 0; j < 32; ++j) {
        uint2 w = *reinterpret_cast<const uint2*>(mine + j * T_BYTES);
        if constexpr (BF) {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(apply_act<ACT>(__uint_as_float(w.x << 16)), apply_act<ACT>(__uint_as_float(w.x & 0xFFFF0000u)));
            const __nv_bfloat162 hi = __floats2bfloat162_rn(apply_act<ACT>(__uint_as_float(w.y << 16)), apply_act<ACT>(__uint_as_float(w.y & 0xFFFF0000u)));
            w.x = *reinterpret_cast<const uint32_t*>(&lo);
            w.y = *reinterpret_cast<const uint32_t*>(&hi);
        } else {
            w.x = __float_as_uint(apply_act<ACT>(__uint_as_float(w.x)));
            w.y = __float_as_uint(apply_act<ACT>(__uint_as_float(w.y)));
        }
        *reinterpret_cast<uint2*>(mine + j * T_BYTES) = w;
    }
}

// Normalisation in place, same ownership as act_slab: RMS y = (x * rstd[row]) * gamma[col], two FP32 products; layer
// normalisation y = ((x - mean[row]) * rstd[row]) * gamma[col] + beta[col], four FP32 operations
// in that order, rounded once to the source dtype.  Rows and columns beyond the tensor hold TMA's zero fill and
// are left alone (their statistics and weights do not exist).
template <bool BF>
__device__ __forceinline__ void norm_slab(uint8_t* mine, const float* __restrict__ rstd, const void* __restrict__ gamma_col,
                                          int rows_here, bool col_ok, const float* __restrict__ mean, const void* __restrict__ beta_col)
{
    if (!col_ok) return;
    auto weights = [](const void* ptr, float (&g)[4]) {
        if constexpr (BF) {
            const uint2 w = *reinterpret_cast<const uint2*>(ptr);
            g[0] = __uint_as_float(w.x << 16); g[1] = __uint_as_float(w.x & 0xFFFF0000u);
            g[2] = __uint_as_float(w.y << 16); g[3] = __uint_as_float(w.y & 0xFFFF0000u);
        } else {
            const float2 w = *reinterpret_cast<const float2*>(ptr);
            g[0] = w.x; g[1] = w.y; g[2] = 0.f; g[3] = 0.f;
        }
    };
    float g[4], b[4] = {0.f, 0.f, 0.f, 0.f};
    weights(gamma_col, g);
    const bool layer = mean != nullptr;      // layer normalisation: subtract the row mean first, add the per-column bias last
    if (layer) weights(beta_col, b);
    // one value: a subtraction (layer normalisation only), two products and an addition (layer normalisation only),
    // each rounded to FP32 on its own (no fused multiply-add: the definition has four roundings)
    auto one = [&](float x, float m, float r, int i) {
        const float t = __fmul_rn(__fmul_rn(layer ? __fsub_rn(x, m) : x, r), g[i]);
        return layer ? __fadd_rn(t, b[i]) : t;
    };
#pragma unroll 8
    for (int j = 0; j < 32; ++j) {
        if (j >= rows_here) break;
        const float r = rstd[j];
        const float m = layer ? mean[j] : 0.f;
        uint2 w = *reinterpret_cast<const uint2*>(mine + j * T_BYTES);
        if constexpr (BF) {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(one(__uint_as_float(w.x << 16), m, r, 0), one(__uint_as_float(w.x & 0xFFFF0000u), m, r, 1));
            const __nv_bfloat162 hi = __floats2bfloat162_rn(one(__uint_as_float(w.y << 16), m, r, 2), one(__uint_as_float(w.y & 0xFFFF0000u), m, r, 3));
            w.x = *reinterpret_cast<const uint32_t*>(&lo);
            w.y = *reinterpret_cast<const uint32_t*>(&hi);
        } else {
            w.x = __float_as_uint(one(__uint_as_float(w.x), m, r, 0));
            w.y = __float_as_uint(one(__uint_as_float(w.y), m, r, 1));
        }
        *reinterpret_cast<uint2*>(mine + j * T_BYTES) = w;
    }
}

// Gated activation in place: gate tile <- act(gate) * up (FP32 product), rounded once to the source dtype.
template <int ACT, bool BF>
__device__ __forceinline__ void glu_slab(uint8_t* gate, const uint8_t* up)
{
#pragma unroll 8
    for (int j = 0; j < 32; ++j) {
        uint2 g = *reinterpret_cast<const uint2*>(gate + j * T_BYTES);
        const uint2 u = *reinterpret_cast<const uint2*>(up + j * T_BYTES);
        if constexpr (BF) {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(apply_act<ACT>(__uint_as_float(g.x << 16)) * __uint_as_float(u.x << 16),
                                                            apply_act<ACT>(__uint_as_float(g.x & 0xFFFF0000u)) * __uint_as_float(u.x & 0xFFFF0000u));
            const __nv_bfloat162 hi = __floats2bfloat162_rn(apply_act<ACT>(__uint_as_float(g.y << 16)) * __uint_as_float(u.y << 16),
                                                            apply_act<ACT>(__uint_as_float(g.y & 0xFFFF0000u)) * __uint_as_float(u.y & 0xFFFF0000u));
            g.x = *reinterpret_cast<const uint32_t*>(&lo);
            g.y = *reinterpret_cast<const uint32_t*>(&hi);
        } else {
            g.x = __float_as_uint(apply_act<ACT>(__uint_as_float(g.x)) * __uint_as_float(u.x));
            g.y = __float_as_uint(apply_act<ACT>(__uint_as_float(g.y)) * __uint_as_float(u.y));
        }
        *reinterpret_cast<uint2*>(gate + j * T_BYTES) = g;
    }
}

// One launch converts up to QT_MAX_TENSORS tensors: their tiles are numbered one tensor after the
// other and dealt out to the CTAs as one pool, so small tensors share one ramp-up and one tail and
// the per-CTA tile counts even out.
constexpr int QT_MAX_TENSORS = 8;
struct QBatch {
    int* status;                          // device status word of the library (bounded waits report here)
    unsigned int* sched;                  // two words owned by the launch's stream, both zero between launches: [0] the next tile to
                                          //   hand out, [1] CTAs that have left; null: tiles are dealt out by CTA index instead
    int test_skip_tile;                   // test builds only: 1 + index of the tile whose load is left out (0 = none)
    int act;                              // MXFP8_ACT_*: applied to every element before the conversion
    const float* rstd;                    // RMS normalisation ahead of the conversion (first tensor only): 1/rms per row,
    const void* gamma;                    //   and the per-column weight in the source dtype; both null when unused
    const float* mean;                    // layer normalisation: the row means (subtracted first) and the per-column bias in the
    const void* beta;                     //   source dtype (added last); both null for RMS normalisation
    int glu_cols;                         // gated activation: the source is [rows, 2 * glu_cols] = (gate | up); 0 when unused
    int up_map;                           // two-source launches: tensor map of the second factor (1), or 0 when it is the up half of the first
    int count;
    int tile_start[QT_MAX_TENSORS + 1];   // first tile of each tensor; [count] = all tiles
    QParams t[QT_MAX_TENSORS];
};
struct QMaps { CUtensorMap m[QT_MAX_TENSORS]; };

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 2^(127 - b) and b for a block with this (finite, non-negative) amax bit pattern.
//   rule_offset = paper_offset<ELEM>() (paper: a mantissa above the largest normal's carries into the exponent = round up)
//               = 0        (ocp: floor)
//   e' = biased exponent after the carry; b = max(e' - emax, 0); 1/X has exponent field 254 - b.
template <int ELEM>
__device__ __forceinline__ uint32_t inv_exp_field(uint32_t amax_bits, uint32_t rule_offset)
{
    const int e = (int)((amax_bits + rule_offset) >> 23);
    return (uint32_t)min(254 + ElemTraits<ELEM>::emax - e, 254);
}

__device__ __forceinline__ uint32_t hmax2_abs(uint32_t a, uint32_t b)
{
    const __nv_bfloat162 x = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&a));
    const __nv_bfloat162 y = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&b));
    const __nv_bfloat162 m = __hmax2(x, y);   // NaN operands are ignored (maxNum)
    return *reinterpret_cast<const uint32_t*>(&m);
}
__device__ __forceinline__ uint32_t hmax2(uint32_t a, uint32_t b)
{
    const __nv_bfloat162 m = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    return *reinterpret_cast<const uint32_t*>(&m);
}
// flags a packed pair of bf16 magnitudes if either half is Inf or NaN
__device__ __forceinline__ uint32_t nonfinite2(uint32_t z) { return (z + 0x00800080u) & 0x80008000u; }

// inv_exp_field for two BF16 amax patterns at once (one per 16-bit half of z, both finite or flagged by the
// caller).  A BF16 pattern is the upper half of the FP32 one, so the rule's offset acts through its upper
// half alone (the lower half of the sum cannot carry), and every step stays inside its 16 bits:
//   e = (h + off16) >> 7 (at most 0x100);  field = min(254 + emax - e, 254), never negative.
template <int ELEM>
__device__ __forceinline__ uint32_t inv_exp_field2(uint32_t z, uint32_t rule_offset16x2)
{
    const uint32_t e2 = ((z + rule_offset16x2) >> 7) & 0x01FF01FFu;
    return __vminu2((254u + ElemTraits<ELEM>::emax) * 0x00010001u - e2, 0x00FE00FEu);
}

// X = 2^(b-127) as FP32 from the exponent field of 1/X (b = 254 - field; b = 0 is the subnormal 2^-127)
__device__ __forceinline__ float scale_from_inv(float inv)
{
    const uint32_t b = 254u - (__float_as_uint(inv) >> 23);
    return __uint_as_float(b ? (b << 23) : 0x00400000u);
}

// 6- and 4-bit codes leave in the layout the tensor cores read (kind::mxf8f6f4): 16 consecutive codes
// of a row form one 16-byte slot, the codes packed as a little-endian bit stream in its first 12
// (6-bit) or 8 (4-bit) bytes, the rest zero.  A slot is 4 lanes wide for a BF16 source (4 codes per
// lane, each lane stores one 32-bit word of the slot) and 8 lanes wide for an FP32 source (2 codes per
// lane, one 16-bit word each).  `c`: this lane's codes, one per byte.  Every lane of the warp calls.
template <int ELEM, int VEC>
__device__ __forceinline__ uint32_t pack_slot(uint32_t c, int lane)
{
    constexpr int B = (ELEM == MXFP8_E2M1) ? 4 : 6;
    if constexpr (VEC == 4) {
        const uint32_t v = (c & 0xFFu) | (((c >> 8) & 0xFFu) << B) | (((c >> 16) & 0xFFu) << (2 * B)) | ((c >> 24) << (3 * B));
        const int j = lane & 3;
        if constexpr (B == 6) {
            // word j of the 96-bit stream = bits 32j.. = (v_j >> 8j) | (v_{j+1} << (24 - 8j)); word 3 is padding
            const uint32_t nxt = __shfl_down_sync(0xFFFFFFFFu, v, 1);
            return j == 3 ? 0u : ((v >> (8 * j)) | (nxt << (24 - 8 * j)));
        } else {
            const uint32_t n1 = __shfl_down_sync(0xFFFFFFFFu, v, 1), n2 = __shfl_down_sync(0xFFFFFFFFu, v, 2);
            return j == 0 ? (v | (n1 << 16)) : (j == 1 ? (n1 | (n2 << 16)) : 0u);
        }
    } else {
        const uint32_t v = (c & 0xFFu) | (((c >> 8) & 0xFFu) << B);
        const int j = lane & 7, base = lane & ~7;
        if constexpr (B == 6) {
            // 16-bit word j of the stream (j < 6) spans the 12-bit values k = 4j/3 and k + 1
            const int k = min((4 * j) / 3, 6);
            const uint32_t lo = __shfl_sync(0xFFFFFFFFu, v, base + k), hi = __shfl_sync(0xFFFFFFFFu, v, base + k + 1);
            return j >= 6 ? 0u : (((lo | (hi << 12)) >> (16 * j - 12 * k)) & 0xFFFFu);
        } else {
            const int k = 2 * (j & 3);
            const uint32_t lo = __shfl_sync(0xFFFFFFFFu, v, base + k), hi = __shfl_sync(0xFFFFFFFFu, v, base + k + 1);
            return j >= 4 ? 0u : (lo | (hi << 8));
        }
    }
}

// One lane's VEC elements of one row: cast x * inv to the element type and store the codes (EMU = false),
// or store the decoded values code * X in the source's own dtype (EMU = true: the MX round trip the
// paper's Hopper runs used, Sec. 3.1).  The decoded product is exact in FP32; BF16 output is one RNE of
// it.  All lanes of the warp call (the sub-byte packing shuffles); only lanes with `store` write.
template <int ELEM, int VEC, bool EMU>
__device__ __forceinline__ void emit(uint8_t* dst, const float (&x)[VEC], const float (&inv)[VEC], const float (&xs)[VEC], int lane,
                                     bool store = true)
{
    constexpr bool SUB = (ELEM != MXFP8_E4M3 && ELEM != MXFP8_E5M2);
    if constexpr (VEC == 4) {
        uint32_t c = cvt_fp8x4<ELEM>(x[0] * inv[0], x[1] * inv[1], x[2] * inv[2], x[3] * inv[3]);
        if constexpr (!EMU) {
            if constexpr (SUB) c = pack_slot<ELEM, VEC>(c, lane);
            if (store) *reinterpret_cast<uint32_t*>(dst) = c;
        } else if (store) {
            const float2 lo = fp8x2_to_float2<ELEM>(c & 0xFFFFu), hi = fp8x2_to_float2<ELEM>(c >> 16);
            const __nv_bfloat162 a = __floats2bfloat162_rn(lo.x * xs[0], lo.y * xs[1]);
            const __nv_bfloat162 b = __floats2bfloat162_rn(hi.x * xs[2], hi.y * xs[3]);
            *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
        }
    } else {
        uint32_t c = cvt_fp8x2<ELEM>(x[0] * inv[0], x[1] * inv[1]);
        if constexpr (!EMU) {
            if constexpr (SUB) c = pack_slot<ELEM, VEC>(c, lane);
            if (store) *reinterpret_cast<uint16_t*>(dst) = (uint16_t)c;
        } else if (store) {
            const float2 f = fp8x2_to_float2<ELEM>(c);
            *reinterpret_cast<float2*>(dst) = make_float2(f.x * xs[0], f.y * xs[1]);
        }
    }
}

// One 32-row slab, fast path: every element finite (checked at the end; the caller reruns the
// slab through slab_careful otherwise), all rows and columns inside the tensor.  Returns
// whether any lane of the warp met an Inf / NaN.
template <int DTYPE, int ELEM, bool DO_ROW, bool DO_COL, bool EMU>
__device__ __forceinline__ bool slab_fast(const uint8_t* __restrict__ my_in, uint8_t* __restrict__ my_qrow,
                                          uint8_t* __restrict__ my_qcol, uint32_t pitch, uint8_t* my_sm_row,
                                          uint8_t* my_sm_col, int lane, uint32_t rule_offset)
{
    constexpr bool BF = (DTYPE == MXFP8_BF16);
    constexpr int VEC = BF ? 4 : 2;
    constexpr int LPB = 32 / VEC;
    uint32_t bad = 0u, zall = 0u;
    const uint32_t rule_offset16x2 = (rule_offset >> 16) * 0x00010001u;
    float col_inv[VEC], col_xs[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) { col_inv[i] = 1.f; col_xs[i] = 1.f; }
    if (DO_COL) {
        uint32_t cbits[VEC];
        if constexpr (BF) {
            uint32_t m0 = 0u, m1 = 0u;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const uint2 w = *reinterpret_cast<const uint2*>(my_in + j * T_BYTES);
                m0 = hmax2(m0, w.x & 0x7FFF7FFFu);     // the running maximum is a magnitude already
                m1 = hmax2(m1, w.y & 0x7FFF7FFFu);
            }
            bad |= nonfinite2(m0) | nonfinite2(m1);
            cbits[0] = m0 << 16; cbits[1] = m0 & 0xFFFF0000u;
            cbits[2] = m1 << 16; cbits[3] = m1 & 0xFFFF0000u;
        } else {
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float2 w = *reinterpret_cast<const float2*>(my_in + j * T_BYTES);
                a0 = fmaxf(a0, fabsf(w.x));
                a1 = fmaxf(a1, fabsf(w.y));
            }
            bad |= (uint32_t)(a0 == INFINITY) | (uint32_t)(a1 == INFINITY);
            cbits[0] = __float_as_uint(a0);
            cbits[1] = __float_as_uint(a1);
        }
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const uint32_t ie = inv_exp_field<ELEM>(cbits[i], rule_offset);
            col_inv[i] = __uint_as_float(ie << 23);
            col_xs[i] = scale_from_inv(col_inv[i]);
            my_sm_col[i * STAGE_PITCH] = (uint8_t)(254u - ie);
        }
    }
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
        float x0[VEC], x1[VEC];
        float inv0 = 1.f, inv1 = 1.f;
        if constexpr (BF) {
            const uint2 w0 = *reinterpret_cast<const uint2*>(my_in + j * T_BYTES);
            const uint2 w1 = *reinterpret_cast<const uint2*>(my_in + (j + 1) * T_BYTES);
            x0[0] = __uint_as_float(w0.x << 16); x0[1] = __uint_as_float(w0.x & 0xFFFF0000u);
            x0[2] = __uint_as_float(w0.y << 16); x0[3] = __uint_as_float(w0.y & 0xFFFF0000u);
            x1[0] = __uint_as_float(w1.x << 16); x1[1] = __uint_as_float(w1.x & 0xFFFF0000u);
            x1[2] = __uint_as_float(w1.y << 16); x1[3] = __uint_as_float(w1.y & 0xFFFF0000u);
            if (DO_ROW) {
                const uint32_t m0 = hmax2_abs(w0.x, w0.y);               // row j  : (max |e0|,|e2| ; max |e1|,|e3|)
                const uint32_t m1 = hmax2_abs(w1.x, w1.y);               // row j+1
                uint32_t z = hmax2(__byte_perm(m0, m1, 0x5410), __byte_perm(m0, m1, 0x7632));   // (amax_j, amax_j+1) of this lane
#pragma unroll
                for (int off = 1; off < LPB; off <<= 1) z = hmax2(z, __shfl_xor_sync(0xFFFFFFFFu, z, off));
                zall = __vmaxu2(zall, z);            // magnitudes order as unsigned integers: finite < Inf < NaN
                const uint32_t ie2 = inv_exp_field2<ELEM>(z, rule_offset16x2);   // both rows' fields, one per half
                inv0 = __uint_as_float(ie2 << 23);
                inv1 = __uint_as_float((ie2 & 0xFFFF0000u) << 7);
                if ((lane & (LPB - 1)) == 0) {
                    const uint32_t sb = 0x00FE00FEu - ie2;
                    my_sm_row[j * STAGE_PITCH] = (uint8_t)sb;
                    my_sm_row[(j + 1) * STAGE_PITCH] = (uint8_t)(sb >> 16);
                }
            }
        } else {
            const float2 w0 = *reinterpret_cast<const float2*>(my_in + j * T_BYTES);
            const float2 w1 = *reinterpret_cast<const float2*>(my_in + (j + 1) * T_BYTES);
            x0[0] = w0.x; x0[1] = w0.y;
            x1[0] = w1.x; x1[1] = w1.y;
            if (DO_ROW) {
                float a0 = fmaxf(fmaxf(fabsf(w0.x), fabsf(w0.y)), 0.f), a1 = fmaxf(fmaxf(fabsf(w1.x), fabsf(w1.y)), 0.f);
#pragma unroll
                for (int off = 1; off < LPB; off <<= 1) {
                    a0 = fmaxf(a0, __shfl_xor_sync(0xFFFFFFFFu, a0, off));
                    a1 = fmaxf(a1, __shfl_xor_sync(0xFFFFFFFFu, a1, off));
                }
                bad |= (uint32_t)(a0 == INFINITY) | (uint32_t)(a1 == INFINITY);
                const uint32_t ie0 = inv_exp_field<ELEM>(__float_as_uint(a0), rule_offset);
                const uint32_t ie1 = inv_exp_field<ELEM>(__float_as_uint(a1), rule_offset);
                inv0 = __uint_as_float(ie0 << 23);
                inv1 = __uint_as_float(ie1 << 23);
                if ((lane & (LPB - 1)) == 0) {
                    my_sm_row[j * STAGE_PITCH] = (uint8_t)(254u - ie0);
                    my_sm_row[(j + 1) * STAGE_PITCH] = (uint8_t)(254u - ie1);
                }
            }
        }
        uint8_t* r0 = my_qrow + (uint64_t)j * pitch;
        uint8_t* c0 = my_qcol + (uint64_t)j * pitch;
        if (DO_ROW) {
            float i0[VEC], i1[VEC], s0[VEC], s1[VEC];
            const float xs0 = EMU ? scale_from_inv(inv0) : 0.f, xs1 = EMU ? scale_from_inv(inv1) : 0.f;
#pragma unroll
            for (int i = 0; i < VEC; ++i) { i0[i] = inv0; i1[i] = inv1; s0[i] = xs0; s1[i] = xs1; }
            emit<ELEM, VEC, EMU>(r0, x0, i0, s0, lane);
            emit<ELEM, VEC, EMU>(r0 + pitch, x1, i1, s1, lane);
        }
        if (DO_COL) {
            emit<ELEM, VEC, EMU>(c0, x0, col_inv, col_xs, lane);
            emit<ELEM, VEC, EMU>(c0 + pitch, x1, col_inv, col_xs, lane);
        }
    }
    return __any_sync(0xFFFFFFFFu, (bad | nonfinite2(zall)) != 0u);
}

// The same slab with everything the fast path leaves out: Inf and NaN elements stay out of
// amax (App. / Sec. 3.3 leaves their handling open; see mxfp8.h), rows and columns outside the
// tensor are not stored.  Rare, so compact rather than fast.
template <int DTYPE, int ELEM, bool DO_ROW, bool DO_COL, bool EMU>
__device__ __noinline__ void slab_careful(const uint8_t* __restrict__ my_in, uint8_t* __restrict__ my_qrow,
                                          uint8_t* __restrict__ my_qcol, uint32_t pitch, uint8_t* my_sm_row,
                                          uint8_t* my_sm_col, int lane, uint32_t rule_offset, int rows_here, bool col_ok)
{
    constexpr bool BF = (DTYPE == MXFP8_BF16);
    constexpr int VEC = BF ? 4 : 2;
    constexpr int LPB = 32 / VEC;
    auto load = [&](int j, float (&x)[VEC]) {
        if constexpr (BF) {
            const uint2 w = *reinterpret_cast<const uint2*>(my_in + j * T_BYTES);
            x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xFFFF0000u);
            x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xFFFF0000u);
        } else {
            const float2 w = *reinterpret_cast<const float2*>(my_in + j * T_BYTES);
            x[0] = w.x; x[1] = w.y;
        }
    };
    float col_inv[VEC], col_xs[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) { col_inv[i] = 1.f; col_xs[i] = 1.f; }
    if (DO_COL) {
        float cmax[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) cmax[i] = 0.f;
#pragma unroll 1
        for (int j = 0; j < 32; ++j) {
            float x[VEC];
            load(j, x);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float a = fabsf(x[i]);
                if (a < INFINITY) cmax[i] = fmaxf(cmax[i], a);   // false for NaN as well
            }
        }
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const uint32_t ie = inv_exp_field<ELEM>(__float_as_uint(cmax[i]), rule_offset);
            col_inv[i] = __uint_as_float(ie << 23);
            col_xs[i] = scale_from_inv(col_inv[i]);
            my_sm_col[i * STAGE_PITCH] = (uint8_t)(254u - ie);
        }
    }
#pragma unroll 1
    for (int j = 0; j < 32; ++j) {
        float x[VEC];
        load(j, x);
        const bool live = col_ok && j < rows_here;
        if (DO_ROW) {
            float m = 0.f;
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float a = fabsf(x[i]);
                if (a < INFINITY) m = fmaxf(m, a);
            }
#pragma unroll
            for (int off = 1; off < LPB; off <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
            const uint32_t ie = inv_exp_field<ELEM>(__float_as_uint(m), rule_offset);
            const float inv = __uint_as_float(ie << 23);
            if ((lane & (LPB - 1)) == 0) my_sm_row[j * STAGE_PITCH] = (uint8_t)(254u - ie);
            if (j < rows_here) {   // warp-uniform; lanes beyond the tensor's last column take part but do not store
                float iv[VEC], sv[VEC];
#pragma unroll
                for (int i = 0; i < VEC; ++i) { iv[i] = inv; sv[i] = scale_from_inv(inv); }
                emit<ELEM, VEC, EMU>(my_qrow + (uint64_t)j * pitch, x, iv, sv, lane, live);
            }
        }
        if (DO_COL && j < rows_here) emit<ELEM, VEC, EMU>(my_qcol + (uint64_t)j * pitch, x, col_inv, col_xs, lane, live);
    }
}

// PRO: what runs on a tile before the conversion.  Separate instantiations, so that the plain conversion carries
// none of the prologue code (folding the prologues in at run time cost the plain kernels 2-5 %).
enum { PRO_NONE = 0, PRO_ELEMENTWISE = 1 /* activation or RMS normalisation */, PRO_GLU = 2 /* gated activation */ };

template <int DTYPE, int ELEM, bool DO_ROW, bool DO_COL, bool EMU, int PRO>
__global__ void __launch_bounds__(QT_THREADS, QT_CTAS_PER_SM)
quantize_tma_kernel(const __grid_constant__ QMaps maps, const __grid_constant__ QBatch batch)
{
    constexpr bool BF = (DTYPE == MXFP8_BF16);
    constexpr int VEC = BF ? 4 : 2;                 // elements per lane per row
    constexpr int T_COLS = T_BYTES / (BF ? 2 : 4);  // 128 or 64
    constexpr int NKB = T_COLS / 32;                // row blocks per tile row: 4 or 2
    constexpr int LPB = 32 / VEC;                   // lanes per row block: 8 or 16
    constexpr bool GLU = (PRO == PRO_GLU);

    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* in_ring = smem;                               // 2 x [128][256]
    uint8_t* sm_scales = smem + RING * IN_BYTES;           // 2 x (row scales + column scales of one tile, 512 bytes each)
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm_scales + 2048);   // [0 .. RING): ring slots; [RING]: the up tile (gated mode)
    uint8_t* up_buf = sm_scales + 2048 + 128;                         // gated mode only: [128][256], allocated by such launches
    const int glu_cols = GLU ? batch.glu_cols : 0;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;   // warp = 32-row slab of the tile
    const uint32_t rule_offset = (batch.t[0].rule == MXFP8_RULE_PAPER) ? paper_offset<ELEM>() : 0u;

    if (tid == 0) {
        for (int k = 0; k < RING; ++k) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[k])));
        if (GLU) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[RING])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int num_tiles = batch.tile_start[batch.count];
    int load_ti = 0;                          // tensor of the tile being loaded (tiles only move forward)
    auto issue_load = [&](int t, int buf) {   // one thread: tile t -> ring slot buf
#ifdef MXFP8_TEST_HOOKS
        if (batch.test_skip_tile && t == batch.test_skip_tile - 1) return;   // never issued: the consumer's bounded wait runs out
#endif
        while (t >= batch.tile_start[load_ti + 1]) ++load_ti;
        int lx, ly;
        divmod((uint32_t)(t - batch.tile_start[load_ti]), (uint32_t)batch.t[load_ti].tiles_x, batch.t[load_ti].tiles_x_magic, ly, lx);
        const uint32_t b = smem_addr(&bars[buf]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)IN_BYTES) : "memory");
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                     ::"r"(smem_addr(in_ring + buf * IN_BYTES)), "l"(&maps.m[load_ti]), "r"(b), "r"(lx * T_COLS), "r"(ly * T_ROWS)
                     : "memory");
    };
    auto issue_up = [&](int t) {              // gated mode (one tensor per launch): the up half of tile t
        int lx, ly;
        divmod((uint32_t)t, (uint32_t)batch.t[0].tiles_x, batch.t[0].tiles_x_magic, ly, lx);
        const uint32_t b = smem_addr(&bars[RING]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)IN_BYTES) : "memory");
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                     ::"r"(smem_addr(up_buf)), "l"(&maps.m[batch.up_map]), "r"(b), "r"(glu_cols + lx * T_COLS), "r"(ly * T_ROWS)
                     : "memory");
    };
    // bounded wait on one of the barriers: false when the limit passed
    auto wait_bar = [&](uint32_t bar, uint32_t parity) {
        uint32_t ok = 0, spins = 0;
        uint64_t t0 = 0;
        while (true) {
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
            if (ok) break;
            if ((++spins & 0xFFu) == 0) {
                uint64_t now;
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                if (t0 == 0) t0 = now;
                else if (now - t0 > QT_WAIT_LIMIT_NS) break;
            }
        }
        return ok != 0;
    };
    // Tiles are handed out in order, one at a time (an atomic counter), as ring slots fall free: whatever the CTAs' relative
    // speed, the tiles in flight stay a compact window of the row-major order, i.e. a few hundred long DRAM rows that all
    // SMs read and write together.  Dealt out by CTA index (tile += gridDim.x) the window widens as soon as the kernel is
    // memory-bound and CTAs drift apart, and the same bytes then move 15 % slower.  Without a counter (batch.sched null)
    // the fixed order serves.
    int* slot_tile = reinterpret_cast<int*>(bars + 8);       // the tile held by (or on its way into) each ring slot
    auto next_tile = [&](int after) {                        // one thread
        return batch.sched ? (int)atomicAdd(batch.sched, 1u) : after + (int)gridDim.x;
    };
    auto leave = [&]() {                                     // one thread, once: the last CTA out zeroes the words for the next launch
        if (batch.sched == nullptr) return;
        __threadfence();
        if (atomicAdd(batch.sched + 1, 1u) == gridDim.x - 1) {
            batch.sched[0] = 0u;
            batch.sched[1] = 0u;
        }
    };
    int tile = 0, ti = 0;
    if (tid == 0) {
        int t = (int)blockIdx.x - (int)gridDim.x;
        for (int k = 0; k < RING; ++k) {
            t = next_tile(t);
            slot_tile[k] = t;
            if (t < num_tiles) issue_load(t, k);
        }
        if (GLU && slot_tile[0] < num_tiles) issue_up(slot_tile[0]);
    }
    __syncthreads();
    for (int it = 0;; ++it) {
        const int buf = it % RING;
        tile = slot_tile[buf];
        if (tile >= num_tiles) break;
        // the tile that will refill this slot: asked for now, needed after the slab (the counter's round trip hides under it);
        // by CTA index it is RING strides on
        int refill = 0;
        if (tid == 0) refill = next_tile(batch.sched ? 0 : tile + (RING - 1) * (int)gridDim.x);
        const uint32_t phase = (uint32_t)(it / RING) & 1u;
        const uint32_t bar_a = smem_addr(&bars[buf]);
        uint8_t* in_tile = in_ring + buf * IN_BYTES;
        uint8_t* sm_row = sm_scales + (it & 1) * 1024;          // 128 rows x 4 blocks, at stage_offset(row)
        uint8_t* sm_col = sm_row + 512;                    // T_COLS columns x 4 blocks, at stage_offset(column)
        while (tile >= batch.tile_start[ti + 1]) ++ti;
        const QParams& p = batch.t[ti];
        int tile_x, tile_y;
        divmod((uint32_t)(tile - batch.tile_start[ti]), (uint32_t)p.tiles_x, p.tiles_x_magic, tile_y, tile_x);
        const int64_t gcol0 = (int64_t)tile_x * T_COLS, grow0 = (int64_t)tile_y * T_ROWS;

        // wait for the tile (bounded: on expiry report through the status word and leave).  A warp needs nothing from the
        // other warps to start on its slab, so the CTA meets only once per tile, at the barrier that frees the ring slot:
        // a warp whose wait ran out skips the tile and says so there.  (The gated mode meets in between for the up tile,
        // so it settles the outcome of the wait first.)
        bool ok = wait_bar(bar_a, phase);
        if constexpr (GLU) ok = wait_bar(smem_addr(&bars[RING]), (uint32_t)it & 1u) && ok;
        ok = __all_sync(0xFFFFFFFFu, ok);
        auto give_up = [&]() {
            if (tid == 0) {
                atomicExch(batch.status, (int)MXFP8_ERR_DEVICE_TIMEOUT);
                leave();
            }
        };
        if constexpr (GLU) {
            if (!__syncthreads_and((int)ok)) { give_up(); return; }
        }
        if (ok) {
        if constexpr (GLU) {
            // gated activation: the slot holds the gate tile, up_buf the up tile; the slot becomes act(gate) * up
            uint8_t* mine = in_tile + warp * 32 * T_BYTES + lane * 8;
            const uint8_t* mine_up = up_buf + warp * 32 * T_BYTES + lane * 8;
            switch (batch.act) {
                case MXFP8_ACT_NONE: glu_slab<MXFP8_ACT_NONE, BF>(mine, mine_up); break;
                case MXFP8_ACT_RELU: glu_slab<MXFP8_ACT_RELU, BF>(mine, mine_up); break;
                case MXFP8_ACT_RELU2: glu_slab<MXFP8_ACT_RELU2, BF>(mine, mine_up); break;
                case MXFP8_ACT_SILU: glu_slab<MXFP8_ACT_SILU, BF>(mine, mine_up); break;
                case MXFP8_ACT_GELU_TANH: glu_slab<MXFP8_ACT_GELU_TANH, BF>(mine, mine_up); break;
                // backward of an activation: the slot holds z, up_buf holds dh; the slot becomes act'(z) * dh
                case ACT_GRAD + MXFP8_ACT_RELU: glu_slab<ACT_GRAD + MXFP8_ACT_RELU, BF>(mine, mine_up); break;
                case ACT_GRAD + MXFP8_ACT_RELU2: glu_slab<ACT_GRAD + MXFP8_ACT_RELU2, BF>(mine, mine_up); break;
                case ACT_GRAD + MXFP8_ACT_SILU: glu_slab<ACT_GRAD + MXFP8_ACT_SILU, BF>(mine, mine_up); break;
                default: glu_slab<ACT_GRAD + MXFP8_ACT_GELU_TANH, BF>(mine, mine_up); break;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();                     // every warp has consumed the up tile: fetch the next one under the conversion
            if (tid == 0 && slot_tile[(it + 1) % RING] < num_tiles) issue_up(slot_tile[(it + 1) % RING]);
        }
        if (PRO == PRO_ELEMENTWISE && batch.rstd != nullptr) {
            // RMS normalisation in place (single-tensor launches only), then the unchanged conversion
            const int64_t row_first = grow0 + warp * 32;
            const int rows_in = (int)max((int64_t)0, min((int64_t)32, p.rows - row_first));
            const int64_t col_first = gcol0 + lane * VEC;
            norm_slab<BF>(in_tile + warp * 32 * T_BYTES + lane * 8, batch.rstd + row_first,
                          static_cast<const uint8_t*>(batch.gamma) + col_first * (BF ? 2 : 4), rows_in, col_first < p.cols,
                          batch.mean ? batch.mean + row_first : nullptr,
                          batch.beta ? static_cast<const uint8_t*>(batch.beta) + col_first * (BF ? 2 : 4) : nullptr);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        if (PRO == PRO_ELEMENTWISE && batch.act != MXFP8_ACT_NONE) {
            // activation in place: every lane rewrites exactly the 8 bytes per row it reads below, rounded once
            // to the source dtype, so what follows equals the conversion of a tensor that holds act(x)
            uint8_t* mine = in_tile + warp * 32 * T_BYTES + lane * 8;
            switch (batch.act) {
                case MXFP8_ACT_RELU: act_slab<MXFP8_ACT_RELU, BF>(mine); break;
                case MXFP8_ACT_RELU2: act_slab<MXFP8_ACT_RELU2, BF>(mine); break;
                case MXFP8_ACT_SILU: act_slab<MXFP8_ACT_SILU, BF>(mine); break;
                default: act_slab<MXFP8_ACT_GELU_TANH, BF>(mine); break;
            }
            // the slot is refilled by a bulk copy later: order these generic-proxy writes before it
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        // this warp's slab: 32 rows; first the fully unrolled fast path (no special values, whole
        // slab inside the tensor), and if it saw an Inf / NaN or the slab is ragged, the careful path
        const uint8_t* my_in = in_tile + warp * 32 * T_BYTES + lane * 8;
        const int64_t my_col = gcol0 + lane * VEC;
        const int rows_here = (int)min((int64_t)32, p.rows - (grow0 + warp * 32));   // rows of this slab inside the tensor
        const bool col_ok = my_col < p.cols;                                         // cols % 16 == 0: a lane's bytes are all in or all out
        // bytes per stored element: 1 (FP8 code), or the source's size when the decoded value is stored
        constexpr int OUT_ESZ = EMU ? (BF ? 2 : 4) : 1;
        uint8_t* my_qrow = p.q_row + ((grow0 + warp * 32) * p.cols + my_col) * OUT_ESZ;
        uint8_t* my_qcol = p.q_col + ((grow0 + warp * 32) * p.cols + my_col) * OUT_ESZ;
        const uint32_t pitch = (uint32_t)p.cols * OUT_ESZ;
        uint8_t* my_sm_row = sm_row + warp * 4 + lane / LPB;                   // row 32 warp + j: + j * STAGE_PITCH
        uint8_t* my_sm_col = sm_col + stage_offset(lane * VEC) + warp;         // column lane * VEC + i: + i * STAGE_PITCH
        const bool whole = __all_sync(0xFFFFFFFFu, col_ok) && rows_here == 32;
        bool special = !whole;
        if (whole)
            special = slab_fast<DTYPE, ELEM, DO_ROW, DO_COL, EMU>(my_in, my_qrow, my_qcol, pitch, my_sm_row, my_sm_col, lane, rule_offset);
        if (special && rows_here > 0)
            slab_careful<DTYPE, ELEM, DO_ROW, DO_COL, EMU>(my_in, my_qrow, my_qcol, pitch, my_sm_row, my_sm_col, lane, rule_offset,
                                                       rows_here, col_ok);
        }

        // every warp is done with this ring slot: refill it with the tile after next
        if (__syncthreads_or((int)!ok)) { give_up(); return; }
        if (tid == 0) {
            slot_tile[buf] = refill;
            if (refill < num_tiles) issue_load(refill, buf);
        }

        // ---- scale bytes (1/32 of the output) leave from the staging arrays ----------
        // A BF16 tile wholly inside the tensor fills exactly one 512-byte atom of the swizzled layout per orientation,
        // and the staging arrays are in the atom's order: one warp stores each atom, 16 bytes per lane.
        if (BF && !EMU && p.sf_layout == MXFP8_SF_SWIZZLED && grow0 + T_ROWS <= p.rows && gcol0 + T_COLS <= p.cols &&
            ((reinterpret_cast<uintptr_t>(p.s_row) | reinterpret_cast<uintptr_t>(p.s_col)) & 15) == 0) {
            if (DO_ROW && warp == 0) {
                const int64_t atoms_k = ((p.cols >> 5) + 3) >> 2;
                *reinterpret_cast<uint4*>(p.s_row + ((int64_t)tile_y * atoms_k + tile_x) * 512 + lane * 16) =
                    *reinterpret_cast<const uint4*>(sm_row + lane * 16);
            }
            if (DO_COL && warp == (DO_ROW ? 1 : 0)) {
                const int64_t atoms_r = ((p.rows >> 5) + 3) >> 2;
                *reinterpret_cast<uint4*>(p.s_col + ((int64_t)tile_x * atoms_r + tile_y) * 512 + lane * 16) =
                    *reinterpret_cast<const uint4*>(sm_col + lane * 16);
            }
            continue;
        }
        // every other tile (ragged, FP32 source, linear layout): one thread per row / per column
        auto first_bytes = [](uint32_t word, int n) { return n >= 4 ? word : (word & ((1u << (8 * max(n, 0))) - 1u)); };
        if (DO_ROW && !EMU && tid < T_ROWS) {
            const int64_t r = grow0 + tid, ncb = p.cols >> 5, kb0 = (int64_t)tile_x * NKB;
            const int nkb = (int)min((int64_t)NKB, ncb - kb0);
            const uint32_t v = r < p.rows ? first_bytes(*reinterpret_cast<const uint32_t*>(sm_row + stage_offset(tid)), nkb) : 0u;
            if (p.sf_layout == MXFP8_SF_SWIZZLED) {
                // every row of a started 128-row atom is written (pad rows / pad K-blocks get 0)
                uint8_t* d = p.s_row + ((int64_t)tile_y * ((ncb + 3) >> 2) + (kb0 >> 2)) * 512 + stage_offset(tid) + (kb0 & 3);
                // a 64-column FP32 tile owns half of the atom's 4 K-blocks; the left half also zeroes
                // the right half when no tile exists there (pad K-blocks)
                if (NKB == 4 || ((kb0 & 3) == 0 && kb0 + NKB >= ncb)) *reinterpret_cast<uint32_t*>(d) = v;
                else *reinterpret_cast<uint16_t*>(d) = (uint16_t)v;
            } else if (r < p.rows) {
                uint8_t* d = p.s_row + r * ncb + kb0;
                for (int kb = 0; kb < nkb; ++kb) d[kb] = (uint8_t)(v >> (8 * kb));
            }
        }
        if (DO_COL && !EMU && tid < T_COLS) {
            const int64_t c = gcol0 + tid, nrb = p.rows >> 5, rb0 = (int64_t)tile_y * 4;
            const int nrb_here = (int)min((int64_t)4, nrb - rb0);
            const uint32_t v = c < p.cols ? first_bytes(*reinterpret_cast<const uint32_t*>(sm_col + stage_offset(tid)), nrb_here) : 0u;
            if (p.sf_layout == MXFP8_SF_SWIZZLED) {
                const int64_t padded_cols = ((p.cols + 127) >> 7) << 7;
                if (c < padded_cols) {
                    *reinterpret_cast<uint32_t*>(p.s_col + ((c >> 7) * ((nrb + 3) >> 2) + tile_y) * 512 + (c & 31) * 16 + ((c >> 5) & 3) * 4) = v;
                    // pad columns no tile covers (FP32 tiles are 64 wide, atoms 128 wide)
                    if (T_COLS == 64 && tile_x == p.tiles_x - 1 && c + 64 >= (int64_t)p.tiles_x * 64 && c + 64 < padded_cols)
                        *reinterpret_cast<uint32_t*>(p.s_col + (((c + 64) >> 7) * ((nrb + 3) >> 2) + tile_y) * 512 + ((c + 64) & 31) * 16 + (((c + 64) >> 5) & 3) * 4) = 0u;
                }
            } else if (c < p.cols) {
                for (int w = 0; w < nrb_here; ++w) p.s_col[(rb0 + w) * p.cols + c] = (uint8_t)(v >> (8 * w));
            }
        }
    }
    if (tid == 0) leave();
}

// Multiprocessors of the current device (looked up once per device)
int qt_sm_count()
{
    static PerDeviceCache<int> cache;
    int n = 0;
    return cache.get(n, [](int dev, int& v) {
               return cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0;
           }) ? n : 0;
}

template <int DTYPE, int ELEM, bool R, bool C, bool EMU, int PRO>
cudaError_t launch(const QMaps& ms, const QBatch& p, cudaStream_t stream)
{
    constexpr bool GLU = (PRO == PRO_GLU);
    constexpr int SMEM = RING * IN_BYTES + 2048 + 128;          // ring, scale staging, barriers
    constexpr int SMEM_USED = GLU ? SMEM + IN_BYTES : SMEM;  // + the up tile of the gated mode
    auto kernel = quantize_tma_kernel<DTYPE, ELEM, R, C, EMU, PRO>;
    static unsigned long long smem_set = 0;
    cudaError_t err = ensure_dynamic_smem(kernel, SMEM_USED, smem_set);
    if (err != cudaSuccess) return err;
    const int tiles = p.tile_start[p.count];
    const int sms = qt_sm_count();
    if (sms <= 0) return cudaErrorInvalidDevice;
    const int max_ctas = sms * (GLU ? 2 : QT_CTAS_PER_SM);
    const int grid = tiles < max_ctas ? tiles : max_ctas;
    kernel<<<grid, QT_THREADS, SMEM_USED, stream>>>(ms, p);
    count_launch(1);
    return cudaGetLastError();
}

template <int DTYPE, int ELEM, bool EMU, int PRO = PRO_NONE>
cudaError_t launch_o(int orientation, const QMaps& ms, const QBatch& p, cudaStream_t st)
{
    if (orientation == MXFP8_ROW) return launch<DTYPE, ELEM, true, false, EMU, PRO>(ms, p, st);
    if (orientation == MXFP8_COL) return launch<DTYPE, ELEM, false, true, EMU, PRO>(ms, p, st);
    return launch<DTYPE, ELEM, true, true, EMU, PRO>(ms, p, st);
}


// All kernels of one element type (source dtypes x orientations x {codes, round trip}); explicitly
// instantiated per element type in the translation units that include this header.
template <int ELEM>
cudaError_t quantize_tma_launch(bool bf16_src, int orientation, bool emulate, const QMaps& ms, const QBatch& p, cudaStream_t st)
{
    if (p.glu_cols || p.up_map)
        return bf16_src ? launch_o<MXFP8_BF16, ELEM, false, PRO_GLU>(orientation, ms, p, st) : launch_o<MXFP8_FP32, ELEM, false, PRO_GLU>(orientation, ms, p, st);
    if (p.rstd != nullptr || p.act != MXFP8_ACT_NONE)
        return bf16_src ? launch_o<MXFP8_BF16, ELEM, false, PRO_ELEMENTWISE>(orientation, ms, p, st)
                        : launch_o<MXFP8_FP32, ELEM, false, PRO_ELEMENTWISE>(orientation, ms, p, st);
    if (emulate)
        return bf16_src ? launch_o<MXFP8_BF16, ELEM, true>(orientation, ms, p, st) : launch_o<MXFP8_FP32, ELEM, true>(orientation, ms, p, st);
    return bf16_src ? launch_o<MXFP8_BF16, ELEM, false>(orientation, ms, p, st) : launch_o<MXFP8_FP32, ELEM, false>(orientation, ms, p, st);
}

}  // namespace
}  // namespace mxfp8
