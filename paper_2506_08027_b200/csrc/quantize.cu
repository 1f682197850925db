// mxfp8_quantize: FP32/BF16 -> MXFP8 in row and/or column blocks from ONE read of the source
// (Sec. 3.2: every tensor is needed blocked along rows and along columns; Sec. 3.3,
// Algorithm 1, App. A.1/A.2: amax -> UE8M0 scale -> RNE saturating cast).
//
// Work decomposition (HBM-bound streaming kernel):
//   CTA tile  = 128 rows x 128 columns = exactly one 512-byte scale atom per orientation.
//   warp tile = 32 rows x (32*VEC) columns held entirely in registers: lane l owns VEC
//               adjacent columns of all 32 rows (VEC = 4 for BF16, 2 for FP32: 8-byte loads,
//               32 of them in flight per thread).
//   column blocks: the 32 rows of a column live in one thread -> amax needs no exchange.
//   row blocks   : 32 columns = 32/VEC adjacent lanes -> amax by xor-shuffles.
//   Q bytes go straight to global memory (each warp store covers whole 32-byte sectors);
//   scale bytes are collected in shared memory in atom order and leave as one 512-byte
//   copy (swizzled layout) or as per-row / per-block-row pieces (linear layout).
#include <atomic>

#include <mutex>

#include "mxfp8_device.cuh"
#include "mxfp8_host.h"

namespace mxfp8 {

namespace {

constexpr int TILE = 128;

template <int DTYPE> struct Src;
template <> struct Src<MXFP8_BF16> {
    static constexpr int VEC = 4;
    using Raw = uint2;
    using Elem = __nv_bfloat16;
    static __device__ __forceinline__ Raw zero() { return make_uint2(0u, 0u); }
    static __device__ __forceinline__ void unpack(const Raw& r, float (&x)[4])
    {
        x[0] = __uint_as_float(r.x << 16);
        x[1] = __uint_as_float(r.x & 0xFFFF0000u);
        x[2] = __uint_as_float(r.y << 16);
        x[3] = __uint_as_float(r.y & 0xFFFF0000u);
    }
    static __device__ __forceinline__ Raw load_scalar(const Elem* p, int n_valid)
    {
        uint32_t h[4] = {0u, 0u, 0u, 0u};
        for (int i = 0; i < 4; ++i)
            if (i < n_valid) h[i] = (uint32_t)__bfloat16_as_ushort(p[i]);
        return make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
    }
};
template <> struct Src<MXFP8_FP32> {
    static constexpr int VEC = 2;
    using Raw = float2;
    using Elem = float;
    static __device__ __forceinline__ Raw zero() { return make_float2(0.f, 0.f); }
    static __device__ __forceinline__ void unpack(const Raw& r, float (&x)[2])
    {
        x[0] = r.x;
        x[1] = r.y;
    }
    static __device__ __forceinline__ Raw load_scalar(const Elem* p, int n_valid)
    {
        return make_float2(n_valid > 0 ? p[0] : 0.f, n_valid > 1 ? p[1] : 0.f);
    }
};

template <int VEC>
__device__ __forceinline__ void store_codes(uint8_t* dst, const uint32_t packed, bool vec_ok, int n_valid)
{
    if (vec_ok) {
        if (VEC == 4) *reinterpret_cast<uint32_t*>(dst) = packed;
        else *reinterpret_cast<uint16_t*>(dst) = (uint16_t)packed;
    } else {
        for (int i = 0; i < VEC; ++i)
            if (i < n_valid) dst[i] = (uint8_t)(packed >> (8 * i));
    }
}

template <int ELEM, int VEC>
__device__ __forceinline__ uint32_t cast_vec(const float (&x)[VEC], const float (&inv)[VEC])
{
    if (VEC == 4) return cvt_fp8x4<ELEM>(x[0] * inv[0], x[1] * inv[1], x[2] * inv[2], x[3] * inv[3]);
    return cvt_fp8x2<ELEM>(x[0] * inv[0], x[1] * inv[1]);
}

// Byte position of (mn, kb) inside one 512-byte scale atom, mn < 128, kb < 4.
__device__ __forceinline__ int atom_pos(int mn, int kb) { return (mn & 31) * 16 + (mn >> 5) * 4 + kb; }

template <int DTYPE, int ELEM, bool DO_ROW, bool DO_COL, bool VEC_OK>
__global__ void __launch_bounds__(128 * (TILE / (32 * Src<DTYPE>::VEC)))
quantize_kernel(const void* __restrict__ src_v, int64_t rows, int64_t cols, int rule, int sf_layout,
                uint8_t* __restrict__ q_row, uint8_t* __restrict__ s_row,
                uint8_t* __restrict__ q_col, uint8_t* __restrict__ s_col, int64_t tiles_x)
{
    using S = Src<DTYPE>;
    constexpr int VEC = S::VEC;
    constexpr int WARP_COLS = 32 * VEC;
    constexpr int WARPS_X = TILE / WARP_COLS;
    constexpr int LPB = 32 / VEC;  // lanes per 32-column row block
    constexpr int THREADS = 128 * WARPS_X;
    const typename S::Elem* __restrict__ src = static_cast<const typename S::Elem*>(src_v);

    __shared__ __align__(16) uint8_t sm_row[512];
    __shared__ __align__(16) uint8_t sm_col[512];

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int wy = warp / WARPS_X;
    const int wx = warp % WARPS_X;
    const int64_t tile_y = (int64_t)blockIdx.x / tiles_x;
    const int64_t tile_x = (int64_t)blockIdx.x % tiles_x;
    const int64_t r0 = tile_y * TILE + wy * 32;
    const int col_in_tile = wx * WARP_COLS + lane * VEC;
    const int64_t c0 = tile_x * TILE + col_in_tile;

    // zero both staging atoms (pad bytes of partial tiles must be 0)
    for (int i = tid; i < 128; i += THREADS) {
        reinterpret_cast<uint32_t*>(sm_row)[i] = 0u;
        reinterpret_cast<uint32_t*>(sm_col)[i] = 0u;
    }
    __syncthreads();

    const int n_valid = (int)max((int64_t)0, min((int64_t)VEC, cols - c0));  // columns this lane owns
    const bool any_col = n_valid > 0;

    // ---- one read of the source: 32 rows x VEC columns per lane ------------------------
    typename S::Raw raw[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const int64_t r = r0 + j;
        raw[j] = S::zero();
        if (r < rows && any_col) {
            const typename S::Elem* p = src + r * cols + c0;
            if (VEC_OK) raw[j] = __ldcs(reinterpret_cast<const typename S::Raw*>(p));
            else raw[j] = S::load_scalar(p, n_valid);
        }
    }

    // ---- column blocks: amax down the 32 rows, all inside this lane ---------------------
    float col_inv[VEC];
    if (DO_COL) {
        float camax[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) camax[i] = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            float x[VEC];
            S::unpack(raw[j], x);
#pragma unroll
            for (int i = 0; i < VEC; ++i) camax[i] = fmaxf(camax[i], fabsf(x[i]));  // NaN ignored
        }
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            if (camax[i] == INFINITY) {  // rare: redo the maximum over finite elements only
                float m = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float x[VEC];
                    S::unpack(raw[j], x);
                    const float a = fabsf(x[i]);
                    if (a < INFINITY) m = fmaxf(m, a);
                }
                camax[i] = m;
            }
            const uint32_t b = scale_byte_from_amax_bits<ELEM>(__float_as_uint(camax[i]), rule);
            col_inv[i] = inv_scale_from_byte(b);
            if (i < n_valid && r0 < rows) sm_col[atom_pos(col_in_tile + i, wy)] = (uint8_t)b;
        }
    }

    // ---- row by row: row-block amax across LPB lanes, then both casts --------------------
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const int64_t r = r0 + j;
        float x[VEC];
        S::unpack(raw[j], x);
        const bool live = (r < rows) && any_col;
        if (DO_ROW) {
            float m = 0.f;
#pragma unroll
            for (int i = 0; i < VEC; ++i) m = fmaxf(m, fabsf(x[i]));  // NaN ignored
#pragma unroll
            for (int off = 1; off < LPB; off <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
            if (__any_sync(0xFFFFFFFFu, m == INFINITY)) {  // rare: finite-only maximum
                m = 0.f;
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    const float a = fabsf(x[i]);
                    if (a < INFINITY) m = fmaxf(m, a);
                }
#pragma unroll
                for (int off = 1; off < LPB; off <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
            }
            const uint32_t b = scale_byte_from_amax_bits<ELEM>(__float_as_uint(m), rule);
            const float inv1 = inv_scale_from_byte(b);
            float inv[VEC];
#pragma unroll
            for (int i = 0; i < VEC; ++i) inv[i] = inv1;
            if (live) {
                store_codes<VEC>(q_row + r * cols + c0, cast_vec<ELEM, VEC>(x, inv), VEC_OK, n_valid);
                if ((lane % LPB) == 0) sm_row[atom_pos(wy * 32 + j, col_in_tile >> 5)] = (uint8_t)b;
            }
        }
        if (DO_COL && live)
            store_codes<VEC>(q_col + r * cols + c0, cast_vec<ELEM, VEC>(x, col_inv), VEC_OK, n_valid);
    }
    __syncthreads();

    // ---- scale bytes leave the CTA ----------------------------------------------------------
    const int64_t tr0 = tile_y * TILE, tc0 = tile_x * TILE;
    if (DO_ROW) {
        const int64_t ncb = cols >> 5;
        if (sf_layout == MXFP8_SF_SWIZZLED) {
            const int64_t atom = tile_y * ((ncb + 3) >> 2) + tile_x;
            if (tid < 32) reinterpret_cast<uint4*>(s_row + atom * 512)[tid] = reinterpret_cast<const uint4*>(sm_row)[tid];
        } else if (tid < TILE && tr0 + tid < rows) {
            uint8_t* d = s_row + (tr0 + tid) * ncb + (tc0 >> 5);
            const int nkb = (int)min((int64_t)4, ncb - (tc0 >> 5));
            if (nkb == 4 && (ncb & 3) == 0) {
                *reinterpret_cast<uint32_t*>(d) = *reinterpret_cast<const uint32_t*>(sm_row + atom_pos(tid, 0));
            } else {
                for (int kb = 0; kb < nkb; ++kb) d[kb] = sm_row[atom_pos(tid, kb)];
            }
        }
    }
    if (DO_COL) {
        const int64_t nrb = rows >> 5;
        if (sf_layout == MXFP8_SF_SWIZZLED) {
            const int64_t atom = tile_x * ((nrb + 3) >> 2) + tile_y;
            if (tid < 32) reinterpret_cast<uint4*>(s_col + atom * 512)[tid] = reinterpret_cast<const uint4*>(sm_col)[tid];
        } else if (tid < TILE && tc0 + tid < cols) {
            const int nrb_here = (int)min((int64_t)4, nrb - (tr0 >> 5));
            for (int w = 0; w < nrb_here; ++w) s_col[((tr0 >> 5) + w) * cols + tc0 + tid] = sm_col[atom_pos(tid, w)];
        }
    }
}

std::atomic<int64_t> g_launches{0};

template <int DTYPE, int ELEM>
cudaError_t launch_quantize(const void* src, int64_t rows, int64_t cols, int orientation, int rule,
                            int sf_layout, uint8_t* q_row, uint8_t* s_row, uint8_t* q_col,
                            uint8_t* s_col, cudaStream_t stream)
{
    constexpr int VEC = Src<DTYPE>::VEC;
    constexpr int THREADS = 128 * (TILE / (32 * VEC));
    const int64_t tiles_x = (cols + TILE - 1) / TILE;
    const int64_t tiles_y = (rows + TILE - 1) / TILE;
    const int64_t tiles = tiles_x * tiles_y;
    if (tiles > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const dim3 grid((unsigned)tiles), block(THREADS);
    const bool vec_ok = (cols % VEC) == 0;
#define MXFP8_LAUNCH(R, C, V) \
    quantize_kernel<DTYPE, ELEM, R, C, V><<<grid, block, 0, stream>>>(src, rows, cols, rule, sf_layout, q_row, s_row, q_col, s_col, tiles_x)
    if (orientation == MXFP8_ROW) MXFP8_LAUNCH(true, false, true);
    else if (orientation == MXFP8_BOTH) MXFP8_LAUNCH(true, true, true);
    else if (vec_ok) MXFP8_LAUNCH(false, true, true);
    else MXFP8_LAUNCH(false, true, false);
#undef MXFP8_LAUNCH
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

}  // namespace

int64_t launches() { return g_launches.load(std::memory_order_relaxed); }
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int quantize_device(const void* src, int src_dtype, int64_t rows, int64_t cols, int orientation,
                    int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col,
                    int sf_layout, cudaStream_t stream)
{
    cudaError_t err;
    uint8_t *qr = static_cast<uint8_t*>(q_row), *sr = static_cast<uint8_t*>(s_row);
    uint8_t *qc = static_cast<uint8_t*>(q_col), *sc = static_cast<uint8_t*>(s_col);
#define MXFP8_ELEM_CASE(E)                                                                                                        \
    case E:                                                                                                                        \
        err = src_dtype == MXFP8_BF16                                                                                              \
                  ? launch_quantize<MXFP8_BF16, E>(src, rows, cols, orientation, scale_rule, sf_layout, qr, sr, qc, sc, stream)   \
                  : launch_quantize<MXFP8_FP32, E>(src, rows, cols, orientation, scale_rule, sf_layout, qr, sr, qc, sc, stream);  \
        break;
    switch (elem) {
        MXFP8_ELEM_CASE(MXFP8_E4M3)
        MXFP8_ELEM_CASE(MXFP8_E5M2)
        default: err = cudaErrorInvalidValue;   // 6- and 4-bit codes are packed 16 to a slot: TMA path only
    }
#undef MXFP8_ELEM_CASE
    return err == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

}  // namespace mxfp8

extern "C" int mxfp8_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                              int orientation, int scale_rule, int elem,
                              void* q_row, void* s_row, void* q_col, void* s_col,
                              int sf_layout, void* stream)
{
    using namespace mxfp8;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!src) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && (!q_row || !s_row)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col || !s_col)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(src)) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_ROW) && (!aligned16(q_row) || !aligned16(s_row))) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_COL) && (!aligned16(q_col) || !aligned16(s_col))) return MXFP8_ERR_ALIGN;
    if (quantize_tma_eligible(src_dtype, rows, cols))
        return quantize_tma_device(src, src_dtype, rows, cols, orientation, scale_rule, elem, q_row, s_row,
                                   q_col, s_col, sf_layout, static_cast<cudaStream_t>(stream));
    if (!fp8_elem(elem)) return MXFP8_ERR_UNSUPPORTED;   // packed 16-code slots need cols % 16 == 0
    return quantize_device(src, src_dtype, rows, cols, orientation, scale_rule, elem, q_row, s_row,
                           q_col, s_col, sf_layout, static_cast<cudaStream_t>(stream));
}

extern "C" int mxfp8_fake_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                                   int orientation, int scale_rule, int elem,
                                   void* dst_row, void* dst_col, void* stream)
{
    using namespace mxfp8;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (!src) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && !dst_row) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && !dst_col) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(src) || ((orientation & MXFP8_ROW) && !aligned16(dst_row)) || ((orientation & MXFP8_COL) && !aligned16(dst_col)))
        return MXFP8_ERR_ALIGN;
    if (!quantize_tma_eligible(src_dtype, rows, cols)) return MXFP8_ERR_UNSUPPORTED;   // needs cols % 16 == 0
    return quantize_tma_device(src, src_dtype, rows, cols, orientation, scale_rule, elem, dst_row, nullptr, dst_col, nullptr,
                               MXFP8_SF_SWIZZLED, static_cast<cudaStream_t>(stream), true);
}

extern "C" int mxfp8_quantize_multi(const mxfp8_quantize_item* items, int count, int src_dtype,
                                    int orientation, int scale_rule, int elem, int sf_layout, void* stream)
{
    using namespace mxfp8;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!items) return MXFP8_ERR_NULL;
    if (count < 1) return MXFP8_ERR_SHAPE;
    if (count > MXFP8_QUANTIZE_MULTI_MAX) return MXFP8_ERR_UNSUPPORTED;
    QuantizeItem batch[MXFP8_QUANTIZE_MULTI_MAX];
    for (int i = 0; i < count; ++i) {
        const mxfp8_quantize_item& it = items[i];
        if (!it.src) return MXFP8_ERR_NULL;
        if ((orientation & MXFP8_ROW) && (!it.q_row || !it.s_row)) return MXFP8_ERR_NULL;
        if ((orientation & MXFP8_COL) && (!it.q_col || !it.s_col)) return MXFP8_ERR_NULL;
        if (it.rows <= 0 || it.cols <= 0) return MXFP8_ERR_SHAPE;
        if ((orientation & MXFP8_ROW) && (it.cols % 32)) return MXFP8_ERR_SHAPE;
        if ((orientation & MXFP8_COL) && (it.rows % 32)) return MXFP8_ERR_SHAPE;
        if (!aligned16(it.src)) return MXFP8_ERR_ALIGN;
        if ((orientation & MXFP8_ROW) && (!aligned16(it.q_row) || !aligned16(it.s_row))) return MXFP8_ERR_ALIGN;
        if ((orientation & MXFP8_COL) && (!aligned16(it.q_col) || !aligned16(it.s_col))) return MXFP8_ERR_ALIGN;
        if (!quantize_tma_eligible(src_dtype, it.rows, it.cols)) return MXFP8_ERR_UNSUPPORTED;   // needs cols % 16 == 0
        batch[i] = QuantizeItem{it.src, it.rows, it.cols, it.q_row, it.s_row, it.q_col, it.s_col};
    }
    return quantize_tma_batch(batch, count, src_dtype, orientation, scale_rule, elem, sf_layout, static_cast<cudaStream_t>(stream));
}

extern "C" int mxfp8_glu_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols, int act,
                                  int orientation, int scale_rule, int elem,
                                  void* q_row, void* s_row, void* q_col, void* s_col,
                                  int sf_layout, void* stream)
{
    using namespace mxfp8;
    if (act < MXFP8_ACT_NONE || act > MXFP8_ACT_GELU_TANH) return MXFP8_ERR_ENUM;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!src) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && (!q_row || !s_row)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col || !s_col)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(src)) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_ROW) && (!aligned16(q_row) || !aligned16(s_row))) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_COL) && (!aligned16(q_col) || !aligned16(s_col))) return MXFP8_ERR_ALIGN;
    // whole tiles along the columns: a tile of the gate half must not reach into the up half
    if (cols % (src_dtype == MXFP8_BF16 ? 128 : 64)) return MXFP8_ERR_UNSUPPORTED;
    if (!quantize_tma_eligible(src_dtype, rows, 2 * cols)) return MXFP8_ERR_UNSUPPORTED;
    const QuantizeItem item{src, rows, cols, q_row, s_row, q_col, s_col};
    return quantize_tma_batch(&item, 1, src_dtype, orientation, scale_rule, elem, sf_layout, static_cast<cudaStream_t>(stream), false, act,
                              nullptr, nullptr, true);
}

namespace mxfp8 {
namespace {
// 1/rms of every row: one warp per row, four 16-byte loads in flight per lane, FP32 accumulation (four lane-strided
// partial sums per lane in a fixed order, then a butterfly), rstd = 1 / sqrt(sum / cols + eps) with IEEE square root
// and division.
template <int DTYPE>
__global__ void __launch_bounds__(256) rms_stats_kernel(const void* __restrict__ src, int64_t rows, int64_t cols, float eps,
                                                        float* __restrict__ rstd)
{
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    constexpr int PER = (DTYPE == MXFP8_BF16) ? 8 : 4;            // elements per 16-byte load
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(src) + row * cols * (DTYPE == MXFP8_BF16 ? 2 : 4));
    const int64_t chunks = cols / PER;
    float part[4] = {0.f, 0.f, 0.f, 0.f};
    auto add = [&](const uint4& w, int k) {
        const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (DTYPE == MXFP8_BF16) {
                const float a = __uint_as_float(u[i] << 16), b = __uint_as_float(u[i] & 0xFFFF0000u);
                part[k] = fmaf(a, a, part[k]);
                part[k] = fmaf(b, b, part[k]);
            } else {
                const float a = __uint_as_float(u[i]);
                part[k] = fmaf(a, a, part[k]);
            }
        }
    };
    int64_t c = lane;
    for (; c + 96 < chunks; c += 128) {          // four 16-byte loads in flight per lane
        const uint4 w0 = p[c], w1 = p[c + 32], w2 = p[c + 64], w3 = p[c + 96];
        add(w0, 0); add(w1, 1); add(w2, 2); add(w3, 3);
    }
    if (c < chunks) { add(p[c], 0); c += 32; }    // up to three 16-byte pieces per lane are left
    if (c < chunks) { add(p[c], 1); c += 32; }
    if (c < chunks) add(p[c], 2);
    float acc = (part[0] + part[1]) + (part[2] + part[3]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if (lane == 0) rstd[row] = 1.0f / sqrtf(acc / (float)cols + eps);
}

// Row statistics of the layer normalisation, one warp per row, as a rule ONE pass: sums of d = x - pivot and of d^2
// with the row's first element as pivot, four 16-byte loads in flight per lane, four partial sums per lane in a fixed
// order, xor butterflies; mean = pivot + S1 / n, rstd = 1 / sqrt((S2 - S1^2 / n) / n + eps) with IEEE square root and
// division.  S2 - S1^2 / n loses log2(1 + (d / sigma)^2) bits when the pivot lies d from the mean: nothing to speak
// of for a pivot within a few standard deviations, everything for an outlier.  So when S1^2 / n takes more than 15/16
// of S2 (the pivot is more than about 4 sigma out, one row in ten thousand of Gaussian data) the row is summed once
// more around the mean just found: the second read comes from cache, and the result is that of a two-pass algorithm.
template <int DTYPE>
__global__ void __launch_bounds__(256) ln_stats_kernel(const void* __restrict__ src, int64_t rows, int64_t cols, float eps,
                                                       float* __restrict__ mean, float* __restrict__ rstd)
{
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    constexpr int PER = (DTYPE == MXFP8_BF16) ? 8 : 4;            // elements per 16-byte load
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(src) + row * cols * (DTYPE == MXFP8_BF16 ? 2 : 4));
    const int64_t chunks = cols / PER;
    const uint32_t first = *reinterpret_cast<const uint32_t*>(p);
    float pivot = (DTYPE == MXFP8_BF16) ? __uint_as_float(first << 16) : __uint_as_float(first);
    float a1 = 0.f, a2 = 0.f;
    const float n = (float)cols;
  for (int pass = 0; pass < 2; ++pass) {
    float s1[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
    auto add = [&](const uint4& w, int k) {
        const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (DTYPE == MXFP8_BF16) {
                const float a = __uint_as_float(u[i] << 16) - pivot, b = __uint_as_float(u[i] & 0xFFFF0000u) - pivot;
                s1[k] += a; s2[k] = fmaf(a, a, s2[k]);
                s1[k] += b; s2[k] = fmaf(b, b, s2[k]);
            } else {
                const float a = __uint_as_float(u[i]) - pivot;
                s1[k] += a; s2[k] = fmaf(a, a, s2[k]);
            }
        }
    };
    int64_t c = lane;
    for (; c + 96 < chunks; c += 128) {
        const uint4 w0 = p[c], w1 = p[c + 32], w2 = p[c + 64], w3 = p[c + 96];
        add(w0, 0); add(w1, 1); add(w2, 2); add(w3, 3);
    }
    if (c < chunks) { add(p[c], 0); c += 32; }    // up to three 16-byte pieces per lane are left
    if (c < chunks) { add(p[c], 1); c += 32; }
    if (c < chunks) add(p[c], 2);
    a1 = (s1[0] + s1[1]) + (s1[2] + s1[3]);
    a2 = (s2[0] + s2[1]) + (s2[2] + s2[3]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        a1 += __shfl_xor_sync(0xFFFFFFFFu, a1, off);
        a2 += __shfl_xor_sync(0xFFFFFFFFu, a2, off);
    }
    // every lane holds the same sums: the decision is uniform over the warp
    if (pass == 1 || !(a1 * a1 / n > 0.9375f * a2)) break;
    pivot = pivot + a1 / n;       // the pivot was far out: once more around the mean
  }
    if (lane == 0) {
        const float var = fmaxf((a2 - a1 * a1 / n) / n, 0.f);
        mean[row] = pivot + a1 / n;
        rstd[row] = 1.0f / sqrtf(var + eps);
    }
}
}  // namespace
}  // namespace mxfp8

extern "C" int mxfp8_layernorm_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                                        const void* gamma, const void* beta, float eps, float* mean, float* rstd,
                                        int orientation, int scale_rule, int elem,
                                        void* q_row, void* s_row, void* q_col, void* s_col,
                                        int sf_layout, void* stream)
{
    using namespace mxfp8;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!src || !gamma || !beta || !mean || !rstd) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && (!q_row || !s_row)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col || !s_col)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0 || !(eps >= 0.f)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(src) || !aligned16(gamma) || !aligned16(beta)) return MXFP8_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(rstd) & 3u) || (reinterpret_cast<uintptr_t>(mean) & 3u)) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_ROW) && (!aligned16(q_row) || !aligned16(s_row))) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_COL) && (!aligned16(q_col) || !aligned16(s_col))) return MXFP8_ERR_ALIGN;
    if (!quantize_tma_eligible(src_dtype, rows, cols)) return MXFP8_ERR_UNSUPPORTED;   // needs cols % 16 == 0
    if ((rows + 7) / 8 > 0x7FFFFFFFLL) return MXFP8_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned blocks = (unsigned)((rows + 7) / 8);
    if (src_dtype == MXFP8_BF16) ln_stats_kernel<MXFP8_BF16><<<blocks, 256, 0, st>>>(src, rows, cols, eps, mean, rstd);
    else ln_stats_kernel<MXFP8_FP32><<<blocks, 256, 0, st>>>(src, rows, cols, eps, mean, rstd);
    count_launch(1);
    if (cudaGetLastError() != cudaSuccess) return MXFP8_ERR_CUDA;
    const QuantizeItem item{src, rows, cols, q_row, s_row, q_col, s_col};
    return quantize_tma_batch(&item, 1, src_dtype, orientation, scale_rule, elem, sf_layout, st, false, MXFP8_ACT_NONE, rstd, gamma, false, mean, beta);
}

namespace mxfp8 {
namespace {
// Argument checks shared by mxfp8_rmsnorm_quantize and its variant with the library's own statistics array.
int rmsnorm_check(const void* src, int src_dtype, int64_t rows, int64_t cols, const void* gamma, float eps, const float* rstd,
                  int orientation, int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col, int sf_layout)
{
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!src || !gamma || !rstd) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && (!q_row || !s_row)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col || !s_col)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0 || !(eps >= 0.f)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(src) || !aligned16(gamma) || (reinterpret_cast<uintptr_t>(rstd) & 3u)) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_ROW) && (!aligned16(q_row) || !aligned16(s_row))) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_COL) && (!aligned16(q_col) || !aligned16(s_col))) return MXFP8_ERR_ALIGN;
    if (!quantize_tma_eligible(src_dtype, rows, cols)) return MXFP8_ERR_UNSUPPORTED;   // needs cols % 16 == 0
    if ((rows + 7) / 8 > 0x7FFFFFFFLL) return MXFP8_ERR_UNSUPPORTED;
    return MXFP8_OK;
}
}  // namespace
}  // namespace mxfp8

extern "C" int mxfp8_rmsnorm_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                                      const void* gamma, float eps, float* rstd,
                                      int orientation, int scale_rule, int elem,
                                      void* q_row, void* s_row, void* q_col, void* s_col,
                                      int sf_layout, void* stream)
{
    using namespace mxfp8;
    const int bad = rmsnorm_check(src, src_dtype, rows, cols, gamma, eps, rstd, orientation, scale_rule, elem, q_row, s_row, q_col, s_col, sf_layout);
    if (bad != MXFP8_OK) return bad;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned blocks = (unsigned)((rows + 7) / 8);
    if (src_dtype == MXFP8_BF16) rms_stats_kernel<MXFP8_BF16><<<blocks, 256, 0, st>>>(src, rows, cols, eps, rstd);
    else rms_stats_kernel<MXFP8_FP32><<<blocks, 256, 0, st>>>(src, rows, cols, eps, rstd);
    count_launch(1);
    if (cudaGetLastError() != cudaSuccess) return MXFP8_ERR_CUDA;
    const QuantizeItem item{src, rows, cols, q_row, s_row, q_col, s_col};
    return quantize_tma_batch(&item, 1, src_dtype, orientation, scale_rule, elem, sf_layout, st, false, MXFP8_ACT_NONE, rstd, gamma);
}

extern "C" int mxfp8_act_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols, int act,
                                  int orientation, int scale_rule, int elem,
                                  void* q_row, void* s_row, void* q_col, void* s_col,
                                  int sf_layout, void* stream)
{
    using namespace mxfp8;
    if (act < MXFP8_ACT_NONE || act > MXFP8_ACT_GELU_TANH) return MXFP8_ERR_ENUM;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    const mxfp8_quantize_item one{src, rows, cols, q_row, s_row, q_col, s_col};
    // same validation as the batched conversion of one tensor
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!src) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && (!q_row || !s_row)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col || !s_col)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(src)) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_ROW) && (!aligned16(q_row) || !aligned16(s_row))) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_COL) && (!aligned16(q_col) || !aligned16(s_col))) return MXFP8_ERR_ALIGN;
    if (!quantize_tma_eligible(src_dtype, rows, cols)) return MXFP8_ERR_UNSUPPORTED;
    const QuantizeItem item{one.src, one.rows, one.cols, one.q_row, one.s_row, one.q_col, one.s_col};
    return quantize_tma_batch(&item, 1, src_dtype, orientation, scale_rule, elem, sf_layout, static_cast<cudaStream_t>(stream), false, act);
}

extern "C" int mxfp8_act_grad_quantize(const void* dh, const void* z, int src_dtype, int64_t rows, int64_t cols, int act,
                                       int orientation, int scale_rule, int elem,
                                       void* q_row, void* s_row, void* q_col, void* s_col,
                                       int sf_layout, void* stream)
{
    using namespace mxfp8;
    if (act < MXFP8_ACT_RELU || act > MXFP8_ACT_GELU_TANH) return MXFP8_ERR_ENUM;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (!dh || !z) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_ROW) && (!q_row || !s_row)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col || !s_col)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_ROW) && (cols % 32)) return MXFP8_ERR_SHAPE;
    if ((orientation & MXFP8_COL) && (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(dh) || !aligned16(z)) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_ROW) && (!aligned16(q_row) || !aligned16(s_row))) return MXFP8_ERR_ALIGN;
    if ((orientation & MXFP8_COL) && (!aligned16(q_col) || !aligned16(s_col))) return MXFP8_ERR_ALIGN;
    if (!quantize_tma_eligible(src_dtype, rows, cols)) return MXFP8_ERR_UNSUPPORTED;   // needs cols % 16 == 0
    // the z tile rides the ring and is overwritten by act'(z) * dh; dh arrives through the second tensor map
    const QuantizeItem item{z, rows, cols, q_row, s_row, q_col, s_col};
    return quantize_tma_batch(&item, 1, src_dtype, orientation, scale_rule, elem, sf_layout, static_cast<cudaStream_t>(stream), false,
                              4 + act, nullptr, nullptr, false, nullptr, nullptr, dh);
}

namespace mxfp8 {
namespace {
// Row statistics of mxfp8_rmsnorm_quantize_static: 65536 rows x 4 bytes = 256 KB that live in the module image.
constexpr int64_t RSTD_STATIC_ROWS = 65536;
static __device__ __align__(256) float g_rstd_static[RSTD_STATIC_ROWS];

// Device address of the array, looked up once per device.
float* rstd_static_address()
{
    static float* addr[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_rstd_static) != cudaSuccess) return nullptr;
        addr[dev] = static_cast<float*>(p);
    }
    return addr[dev];
}
}  // namespace
}  // namespace mxfp8

extern "C" int64_t mxfp8_rmsnorm_quantize_static_max_rows(void) { return mxfp8::RSTD_STATIC_ROWS; }

extern "C" int mxfp8_rmsnorm_quantize_static(const void* src, int src_dtype, int64_t rows, int64_t cols,
                                             const void* gamma, float eps,
                                             int orientation, int scale_rule, int elem,
                                             void* q_row, void* s_row, void* q_col, void* s_col,
                                             int sf_layout, void* stream)
{
    using namespace mxfp8;
    // the same checks, in the same order, as the call with a caller's buffer (the array stands in for it: any aligned
    // non-null address passes those two checks); then this variant's own limit; only then the device is asked
    const int bad = rmsnorm_check(src, src_dtype, rows, cols, gamma, eps, reinterpret_cast<const float*>(uintptr_t(256)), orientation,
                                  scale_rule, elem, q_row, s_row, q_col, s_col, sf_layout);
    if (bad != MXFP8_OK) return bad;
    if (rows > RSTD_STATIC_ROWS) return MXFP8_ERR_UNSUPPORTED;
    float* rstd = rstd_static_address();      // the array of the device that is current on this thread
    if (!rstd) return MXFP8_ERR_CUDA;
    return mxfp8_rmsnorm_quantize(src, src_dtype, rows, cols, gamma, eps, rstd, orientation, scale_rule, elem,
                                  q_row, s_row, q_col, s_col, sf_layout, stream);
}
