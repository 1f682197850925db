// mxfp8_dequantize: decoded value Q_i * X (Sec. 2) written as FP32 or BF16.
//
// Every FP8 value times a power of two has at most 4 significant bits and magnitude at
// least 2^-136, so the FP32 product below is exact (or overflows to infinity exactly where
// the real product exceeds the FP32 range); the BF16 result is one RNE rounding of it.
#include "mxfp8_device.cuh"
#include "mxfp8_host.h"

namespace mxfp8 {
namespace {

// X = 2^(b-127) as FP32: b = 0 is the subnormal 2^-127, b = 255 is NaN.
__device__ __forceinline__ float scale_value(uint32_t b)
{
    if (b == 0xFFu) return __uint_as_float(0x7FC00000u);
    return (b == 0u) ? __uint_as_float(0x00400000u) : __uint_as_float(b << 23);
}

template <int ELEM, int DST, int ORIENT>
__global__ void __launch_bounds__(256)
dequantize_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ s, int64_t rows, int64_t cols,
                  int sf_layout, void* __restrict__ dst_v, int64_t chunks_per_row)
{
    // one thread = 16 consecutive elements of a row (or the ragged tail of the row)
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * chunks_per_row) return;
    const int64_t r = idx / chunks_per_row;
    const int64_t c0 = (idx % chunks_per_row) * 16;
    const int n = (int)min((int64_t)16, cols - c0);
    const bool vec = (n == 16) && ((cols & 15) == 0);

    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (vec) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(q + r * cols + c0));
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else {
        for (int i = 0; i < n; ++i) w[i >> 2] |= (uint32_t)q[r * cols + c0 + i] << (8 * (i & 3));
    }

    if constexpr (ELEM != MXFP8_E4M3 && ELEM != MXFP8_E5M2) {
        // 6- and 4-bit codes arrive as one packed 16-byte slot (little-endian bit stream in the first
        // 12 / 8 bytes): spread them to one code per byte
        constexpr int B = (ELEM == MXFP8_E2M1) ? 4 : 6;
        const uint32_t st[4] = {w[0], w[1], w[2], 0u};
        uint32_t u[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int bit = B * i, wd = bit >> 5, off = bit & 31;
            uint32_t code = st[wd] >> off;
            if (off + B > 32) code |= st[wd + 1] << (32 - off);
            u[i >> 2] |= (code & ((1u << B) - 1u)) << (8 * (i & 3));
        }
        w[0] = u[0]; w[1] = u[1]; w[2] = u[2]; w[3] = u[3];
    }

    float out[16];
    float row_scale = 0.f;
    if (ORIENT == MXFP8_ROW) {
        const int64_t ncb = cols >> 5, kb = c0 >> 5;
        const int64_t off = (sf_layout == MXFP8_SF_SWIZZLED) ? sf_swizzled_offset(r, kb, ncb) : r * ncb + kb;
        row_scale = scale_value(s[off]);
    }
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        const float2 f = fp8x2_to_float2<ELEM>((w[p >> 1] >> (16 * (p & 1))) & 0xFFFFu);
        float s0 = row_scale, s1 = row_scale;
        if (ORIENT == MXFP8_COL) {
            const int64_t nrb = rows >> 5, kb = r >> 5;
            const int64_t ca = c0 + 2 * p, cb = c0 + 2 * p + 1;
            if (2 * p < n)
                s0 = scale_value(s[(sf_layout == MXFP8_SF_SWIZZLED) ? sf_swizzled_offset(ca, kb, nrb) : kb * cols + ca]);
            if (2 * p + 1 < n)
                s1 = scale_value(s[(sf_layout == MXFP8_SF_SWIZZLED) ? sf_swizzled_offset(cb, kb, nrb) : kb * cols + cb]);
        }
        out[2 * p] = f.x * s0;
        out[2 * p + 1] = f.y * s1;
    }

    if (DST == MXFP8_FP32) {
        float* d = static_cast<float*>(dst_v) + r * cols + c0;
        if (vec) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                reinterpret_cast<float4*>(d)[i] = make_float4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
        } else {
            for (int i = 0; i < n; ++i) d[i] = out[i];
        }
    } else {
        __nv_bfloat16* d = static_cast<__nv_bfloat16*>(dst_v) + r * cols + c0;
        if (vec) {
            uint32_t pk[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(out[2 * i], out[2 * i + 1]);
                pk[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
            reinterpret_cast<uint4*>(d)[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            reinterpret_cast<uint4*>(d)[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        } else {
            for (int i = 0; i < n; ++i) d[i] = __float2bfloat16_rn(out[i]);
        }
    }
}

// Fast path (cols % 128 == 0): a warp step covers 128 consecutive elements of one row; lane l owns
// elements 4l..4l+3, so the loads (4 bytes per lane) and the stores (16 bytes FP32 / 8 bytes BF16
// per lane) of a warp are contiguous.  Each warp takes UNROLL consecutive steps with all its loads
// issued before the first use.
template <int ELEM, int DST, int ORIENT>
__global__ void __launch_bounds__(256)
dequantize_vec_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ s, int64_t rows, int64_t cols,
                      int sf_layout, void* __restrict__ dst_v, int64_t groups)
{
    constexpr int UNROLL = 8;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t g0 = warp * UNROLL;
    if (g0 >= groups) return;
    const int64_t groups_per_row = cols >> 7;
    uint32_t w[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u)
        w[u] = (g0 + u < groups) ? __ldcs(reinterpret_cast<const uint32_t*>(q) + (g0 + u) * 32 + lane) : 0u;
    int64_t r = g0 / groups_per_row;                       // one division per warp, then step
    int64_t cg = g0 - r * groups_per_row;
#pragma unroll
    for (int u = 0; u < UNROLL; ++u, ++cg) {
        if (g0 + u >= groups) break;
        if (cg == groups_per_row) { cg = 0; ++r; }
        const int64_t c = cg * 128 + lane * 4;
        float sc[4];
        if (ORIENT == MXFP8_ROW) {
            const int64_t ncb = cols >> 5, kb = c >> 5;
            const float v = scale_value(s[(sf_layout == MXFP8_SF_SWIZZLED) ? sf_swizzled_offset(r, kb, ncb) : r * ncb + kb]);
            sc[0] = sc[1] = sc[2] = sc[3] = v;
        } else {
            const int64_t nrb = rows >> 5, kb = r >> 5;
            if (sf_layout == MXFP8_SF_SWIZZLED) {
                const uint8_t* base = s + sf_swizzled_offset(c, kb, nrb);   // columns c..c+3 share the atom: 16 bytes apart
#pragma unroll
                for (int i = 0; i < 4; ++i) sc[i] = scale_value(base[i * 16]);
            } else {
                const uint32_t four = *reinterpret_cast<const uint32_t*>(s + kb * cols + c);
#pragma unroll
                for (int i = 0; i < 4; ++i) sc[i] = scale_value((four >> (8 * i)) & 0xFFu);
            }
        }
        const float2 lo = fp8x2_to_float2<ELEM>(w[u] & 0xFFFFu), hi = fp8x2_to_float2<ELEM>(w[u] >> 16);
        const float o0 = lo.x * sc[0], o1 = lo.y * sc[1], o2 = hi.x * sc[2], o3 = hi.y * sc[3];
        if (DST == MXFP8_FP32) {
            __stcs(reinterpret_cast<float4*>(static_cast<float*>(dst_v) + r * cols + c), make_float4(o0, o1, o2, o3));
        } else {
            const __nv_bfloat162 a = __floats2bfloat162_rn(o0, o1), b2 = __floats2bfloat162_rn(o2, o3);
            __stcs(reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(dst_v) + r * cols + c),
                   make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b2)));
        }
    }
}

// Four decoded elements of one lane: codes -> FP32 (exact), times the scales, one rounding if BF16 is asked.
template <int ELEM, int DST>
__device__ __forceinline__ void decode_store4(uint32_t codes, float s0, float s1, float s2, float s3, void* dst_elem)
{
    const float2 lo = fp8x2_to_float2<ELEM>(codes & 0xFFFFu), hi = fp8x2_to_float2<ELEM>(codes >> 16);
    const float o0 = lo.x * s0, o1 = lo.y * s1, o2 = hi.x * s2, o3 = hi.y * s3;
    if (DST == MXFP8_FP32) {
        __stcs(reinterpret_cast<float4*>(dst_elem), make_float4(o0, o1, o2, o3));
    } else {
        const __nv_bfloat162 a = __floats2bfloat162_rn(o0, o1), b2 = __floats2bfloat162_rn(o2, o3);
        __stcs(reinterpret_cast<uint2*>(dst_elem), make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b2)));
    }
}

// Row blocks, cols % 1024 == 0: a warp owns 1024 consecutive elements of one row = 32 blocks.  Lane l fetches
// and decodes the scale of block l once; in step u (128 elements) lane l owns elements 4l..4l+3 of block
// 4u + l/8 and takes its scale by shuffle.  One 4-byte load and one 8/16-byte store per lane and step.
template <int ELEM, int DST>
__global__ void __launch_bounds__(256)
dequantize_row1024_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ s, int64_t cols, int sf_layout,
                          void* __restrict__ dst_v, int64_t chunks)
{
    const int lane = threadIdx.x & 31;
    const int64_t chunk = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;     // 1024-element chunk
    if (chunk >= chunks) return;
    const int64_t per_row = cols >> 10;
    const int64_t r = chunk / per_row;
    const int64_t c0 = (chunk - r * per_row) << 10;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(q + r * cols + c0) + lane;
    uint32_t w[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) w[u] = __ldcs(src + u * 32);
    const int64_t ncb = cols >> 5, kb = (c0 >> 5) + lane;
    const float mine = scale_value(s[(sf_layout == MXFP8_SF_SWIZZLED) ? sf_swizzled_offset(r, kb, ncb) : r * ncb + kb]);
    constexpr int ESZ = (DST == MXFP8_FP32) ? 4 : 2;
    uint8_t* out = static_cast<uint8_t*>(dst_v) + (r * cols + c0 + lane * 4) * ESZ;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const float sc = __shfl_sync(0xFFFFFFFFu, mine, 4 * u + (lane >> 3));
        decode_store4<ELEM, DST>(w[u], sc, sc, sc, sc, out + u * 128 * ESZ);
    }
}

// Column blocks: a warp owns a strip of 128 columns x 32 rows = one block of every column of the strip, so
// each lane fetches and decodes the four scales of its columns once and reuses them for the 32 rows.
template <int ELEM, int DST>
__global__ void __launch_bounds__(256)
dequantize_colstrip_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ s, int64_t rows, int64_t cols,
                           int sf_layout, void* __restrict__ dst_v, int64_t strips)
{
    const int lane = threadIdx.x & 31;
    const int64_t strip = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (strip >= strips) return;
    const int64_t strips_per_band = cols >> 7;
    const int64_t kb = strip / strips_per_band;                       // 32-row band = block index along the rows
    const int64_t c = ((strip - kb * strips_per_band) << 7) + lane * 4;
    const int64_t nrb = rows >> 5;
    float sc[4];
    if (sf_layout == MXFP8_SF_SWIZZLED) {
        const uint8_t* base = s + sf_swizzled_offset(c, kb, nrb);    // columns c..c+3 sit 16 bytes apart in their atom
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[i] = scale_value(base[i * 16]);
    } else {
        const uint32_t four = *reinterpret_cast<const uint32_t*>(s + kb * cols + c);
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[i] = scale_value((four >> (8 * i)) & 0xFFu);
    }
    constexpr int ESZ = (DST == MXFP8_FP32) ? 4 : 2;
    const uint8_t* src = q + (kb * 32) * cols + c;
    uint8_t* out = static_cast<uint8_t*>(dst_v) + ((kb * 32) * cols + c) * ESZ;
#pragma unroll
    for (int j0 = 0; j0 < 32; j0 += 8) {
        uint32_t w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) w[j] = __ldcs(reinterpret_cast<const uint32_t*>(src + (int64_t)(j0 + j) * cols));
#pragma unroll
        for (int j = 0; j < 8; ++j) decode_store4<ELEM, DST>(w[j], sc[0], sc[1], sc[2], sc[3], out + (int64_t)(j0 + j) * cols * ESZ);
    }
}

template <int ELEM, int DST, int ORIENT>
cudaError_t launch(const uint8_t* q, const uint8_t* s, int64_t rows, int64_t cols, int sf_layout,
                   void* dst, cudaStream_t stream)
{
    if constexpr (ELEM == MXFP8_E4M3 || ELEM == MXFP8_E5M2) {
        if (ORIENT == MXFP8_ROW && (cols & 1023) == 0) {
            const int64_t chunks = rows * (cols >> 10);
            const int64_t blocks = (chunks + 7) / 8;               // 8 warps per block
            if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
            dequantize_row1024_kernel<ELEM, DST><<<(unsigned)blocks, 256, 0, stream>>>(q, s, cols, sf_layout, dst, chunks);
            count_launch(1);
            return cudaGetLastError();
        }
        if (ORIENT == MXFP8_COL && (cols & 127) == 0) {
            const int64_t strips = (rows >> 5) * (cols >> 7);
            const int64_t blocks = (strips + 7) / 8;
            if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
            dequantize_colstrip_kernel<ELEM, DST><<<(unsigned)blocks, 256, 0, stream>>>(q, s, rows, cols, sf_layout, dst, strips);
            count_launch(1);
            return cudaGetLastError();
        }
    }
    if constexpr (ELEM == MXFP8_E4M3 || ELEM == MXFP8_E5M2) if ((cols & 127) == 0) {
        const int64_t groups = rows * (cols / 128);            // warp steps of 128 elements
        const int64_t warps = (groups + 7) / 8;
        const int64_t blocks = (warps + 7) / 8;                // 8 warps per block
        if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
        dequantize_vec_kernel<ELEM, DST, ORIENT><<<(unsigned)blocks, 256, 0, stream>>>(q, s, rows, cols, sf_layout, dst, groups);
        count_launch(1);
        return cudaGetLastError();
    }
    const int64_t chunks = (cols + 15) / 16;
    const int64_t blocks = (rows * chunks + 255) / 256;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    dequantize_kernel<ELEM, DST, ORIENT><<<(unsigned)blocks, 256, 0, stream>>>(q, s, rows, cols, sf_layout, dst, chunks);
    count_launch(1);
    return cudaGetLastError();
}

template <int ELEM, int DST>
cudaError_t launch_o(int orient, const uint8_t* q, const uint8_t* s, int64_t rows, int64_t cols,
                     int sf_layout, void* dst, cudaStream_t stream)
{
    return orient == MXFP8_ROW ? launch<ELEM, DST, MXFP8_ROW>(q, s, rows, cols, sf_layout, dst, stream)
                               : launch<ELEM, DST, MXFP8_COL>(q, s, rows, cols, sf_layout, dst, stream);
}

}  // namespace
}  // namespace mxfp8

extern "C" int mxfp8_dequantize(const void* q, const void* s, int64_t rows, int64_t cols,
                                int orientation, int elem, int sf_layout,
                                void* dst, int dst_dtype, void* stream)
{
    using namespace mxfp8;
    if (orientation != MXFP8_ROW && orientation != MXFP8_COL) return MXFP8_ERR_ENUM;
    if (!valid_elem(elem)) return MXFP8_ERR_ENUM;
    if (sf_layout != MXFP8_SF_LINEAR && sf_layout != MXFP8_SF_SWIZZLED) return MXFP8_ERR_ENUM;
    if (dst_dtype != MXFP8_FP32 && dst_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (!q || !s || !dst) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if (orientation == MXFP8_ROW ? (cols % 32) : (rows % 32)) return MXFP8_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(s) || !aligned16(dst)) return MXFP8_ERR_ALIGN;
    if (!fp8_elem(elem) && (cols % 16)) return MXFP8_ERR_UNSUPPORTED;   // packed 16-code slots
    const uint8_t* qq = static_cast<const uint8_t*>(q);
    const uint8_t* ss = static_cast<const uint8_t*>(s);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t err;
#define MXFP8_ELEM_CASE(E)                                                                                               \
    case E:                                                                                                               \
        err = dst_dtype == MXFP8_FP32 ? launch_o<E, MXFP8_FP32>(orientation, qq, ss, rows, cols, sf_layout, dst, st)     \
                                      : launch_o<E, MXFP8_BF16>(orientation, qq, ss, rows, cols, sf_layout, dst, st);    \
        break;
    switch (elem) {
        MXFP8_ELEM_CASE(MXFP8_E4M3)
        MXFP8_ELEM_CASE(MXFP8_E5M2)
        MXFP8_ELEM_CASE(MXFP8_E2M3)
        MXFP8_ELEM_CASE(MXFP8_E3M2)
        MXFP8_ELEM_CASE(MXFP8_E2M1)
        default: err = cudaErrorInvalidValue;
    }
#undef MXFP8_ELEM_CASE
    return err == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}
