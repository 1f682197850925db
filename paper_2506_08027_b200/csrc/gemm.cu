// mxfp8_gemm: block-scaled MXFP8 matrix product on the 5th-generation tensor cores
// (Sec. 2 and App. A.3: per 32-element block dot product of the FP8 elements, scaled by the
// two blocks' UE8M0 scales, accumulated in FP32).
//
// Structure (one persistent CTA per SM, 192 threads, warp-specialised):
//   warp 0      TMA producer: A/B tiles (128-byte swizzle) and 512-byte scale atoms -> smem ring
//   warp 1      MMA issuer (one thread): tcgen05.cp scales smem->TMEM, then
//               tcgen05.mma.kind::mxf8f6f4.block_scale over the K loop; owns TMEM alloc/dealloc
//   warps 2..5  epilogue: tcgen05.ld the FP32 accumulator from TMEM, convert, store D
//   A CTA tile is 128 x BN (BN = 256 or 128) with K step 128 (= 4 MMAs of K = 32, one scale
//   byte per row per MMA = one 4-byte TMEM column entry per K step).
//   Every mbarrier wait is bounded: on expiry the kernel records MXFP8_ERR_DEVICE_TIMEOUT in
//   the device status word, raises an abort flag that all roles poll, drains and exits.
#include <cuda.h>

#include "mxfp8_device.cuh"
#include "mxfp8_host.h"

namespace mxfp8 {

__device__ int g_device_status = 0;

int read_and_clear_device_status(cudaStream_t stream)
{
    if (cudaStreamSynchronize(stream) != cudaSuccess) return MXFP8_ERR_CUDA;
    int h = 0, z = 0;
    if (cudaMemcpyFromSymbol(&h, g_device_status, sizeof(int)) != cudaSuccess) return MXFP8_ERR_CUDA;
    if (h != 0 && cudaMemcpyToSymbol(g_device_status, &z, sizeof(int)) != cudaSuccess) return MXFP8_ERR_CUDA;
    return h == 0 ? MXFP8_OK : MXFP8_ERR_DEVICE_TIMEOUT;
}

namespace {

constexpr int BM = 128;            // tile rows (TMEM lanes)
constexpr int BK = 128;            // K bytes per pipeline stage = one 128-byte swizzle row
constexpr int GEMM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;  // bounded waits give up after 2 s

struct GemmParams {
    int64_t M, N, K;
    int a_mn, b_mn;       // 1 = MN-major storage
    int a_elem, b_elem;
    int out_dtype;
    int tiles_m, tiles_n, num_tiles, num_kb;
};

template <int BN> struct Cfg {
    static constexpr int ACC_STAGES = (BN == 256) ? 1 : 2;
    static constexpr int STAGES = (BN == 256) ? 4 : 6;
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int SFB_ATOMS = BN / 128;
    static constexpr int SF_COLS = 4 + 4 * SFB_ATOMS;          // TMEM columns of scales per stage
    static constexpr int SF_COL0 = ACC_STAGES * BN;            // first scale column
    static constexpr uint32_t STAGE_TX = A_BYTES + B_BYTES + 512 + 512 * SFB_ATOMS;
    static constexpr int SMEM_A = 0;
    static constexpr int SMEM_B = SMEM_A + STAGES * A_BYTES;
    static constexpr int SMEM_SFA = SMEM_B + STAGES * B_BYTES;
    static constexpr int SMEM_SFB = SMEM_SFA + STAGES * 512;
    static constexpr int SMEM_BAR = SMEM_SFB + STAGES * 512 * SFB_ATOMS;
    static constexpr int NUM_BARS = 2 * STAGES + 2 * ACC_STAGES + 1;
    static constexpr int SMEM_MISC = SMEM_BAR + NUM_BARS * 8;  // tmem pointer, abort flag
    static constexpr int SMEM_TOTAL = SMEM_MISC + 16 + 1024;   // + slack to align the base to 1024
    static_assert(SF_COL0 + STAGES * SF_COLS <= TMEM_COLS, "TMEM budget");
};

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ uint64_t global_timer()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when the abort flag is up or the time limit passed (the latter also
// records the timeout and raises the flag for the other roles).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    uint32_t spins = 0;
    uint64_t t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xFFu) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                atomicExch(&g_device_status, (int)MXFP8_ERR_DEVICE_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t desc)
{
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte
// offsets in 16-byte units, version 1, swizzle mode in bits 61-63 (2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}

// Block-scaled instruction descriptor: element formats, majorness, N>>3, UE8M0 scales, M>>4.
__device__ __forceinline__ uint32_t make_idesc(int a_elem, int b_elem, int a_mn, int b_mn, int n)
{
    return ((uint32_t)a_elem << 7) | ((uint32_t)b_elem << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(BM >> 4) << 24);
}

template <int BN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const uint8_t* __restrict__ sfa, const uint8_t* __restrict__ sfb, void* __restrict__ D,
            const GemmParams p)
{
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;   // 128-byte swizzle needs 1024-byte alignment
    uint8_t* base_ptr = smem_raw + (base - raw_addr);

    const uint32_t bar0 = base + C::SMEM_BAR;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (C::STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * C::STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * C::STAGES + C::ACC_STAGES + a); };
    const uint32_t drain_bar = bar0 + 8u * (2 * C::STAGES + 2 * C::ACC_STAGES);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + C::SMEM_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::SMEM_MISC + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < C::ACC_STAGES; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int64_t atoms_k = p.K >> 7;   // scale atoms along K (4 K-blocks each)

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
                const int m0 = tm * BM, n0 = tn * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = full_bar(s);
                    mbar_expect_tx(fb, C::STAGE_TX);
                    const uint32_t sa = base + C::SMEM_A + s * C::A_BYTES;
                    const uint32_t sb = base + C::SMEM_B + s * C::B_BYTES;
                    const int k0 = kb * BK;
                    if (!p.a_mn) tma_load_2d(sa, &tmap_a, fb, k0, m0);
                    else tma_load_2d(sa, &tmap_a, fb, m0, k0);
                    if (!p.b_mn) {
                        tma_load_2d(sb, &tmap_b, fb, k0, n0);
                    } else {
#pragma unroll
                        for (int j = 0; j < C::SFB_ATOMS; ++j) tma_load_2d(sb + j * 16384, &tmap_b, fb, n0 + j * 128, k0);
                    }
                    bulk_load(base + C::SMEM_SFA + s * 512, sfa + ((int64_t)tm * atoms_k + kb) * 512, 512, fb);
#pragma unroll
                    for (int j = 0; j < C::SFB_ATOMS; ++j)
                        bulk_load(base + C::SMEM_SFB + (s * C::SFB_ATOMS + j) * 512,
                                  sfb + ((int64_t)(tn * C::SFB_ATOMS + j) * atoms_k + kb) * 512, 512, fb);
                }
            }
            if (!ok) {
                // give copies already in flight time to land before the CTA's smem is released
                for (int i = 0; i < 200; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc0 = make_idesc(p.a_elem, p.b_elem, p.a_mn, p.b_mn, BN);
            uint32_t it = 0, acc_it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++acc_it) {
                const int as = acc_it % C::ACC_STAGES;
                const uint32_t aph = (acc_it / C::ACC_STAGES) & 1u;
                if (!mbar_wait(tempty_bar(as), aph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sfa_t = tmem_base + C::SF_COL0 + s * C::SF_COLS;
                    const uint32_t sfb_t = sfa_t + 4;
                    // scales: 32 rows x 16 bytes per atom, no swizzle, 8-row groups 128 bytes apart
                    tc_cp_sf(sfa_t, smem_desc(base + C::SMEM_SFA + s * 512, 0, 128, 0));
#pragma unroll
                    for (int j = 0; j < C::SFB_ATOMS; ++j)
                        tc_cp_sf(sfb_t + 4 * j, smem_desc(base + C::SMEM_SFB + (s * C::SFB_ATOMS + j) * 512, 0, 128, 0));
                    const uint32_t sa = base + C::SMEM_A + s * C::A_BYTES;
                    const uint32_t sb = base + C::SMEM_B + s * C::B_BYTES;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        // K-major: 32 bytes further along the swizzled row; 8-row groups 1024 B apart.
                        // MN-major: 32 K-rows (4096 B) further; 8-K-row groups 1024 B apart, 128-wide
                        // MN slabs 16384 B apart.
                        const uint64_t ad = p.a_mn ? smem_desc(sa + k * 4096, 16384, 1024, 2) : smem_desc(sa + k * 32, 0, 1024, 2);
                        const uint64_t bd = p.b_mn ? smem_desc(sb + k * 4096, 16384, 1024, 2) : smem_desc(sb + k * 32, 0, 1024, 2);
                        const uint32_t idesc = idesc0 | ((uint32_t)k << 29) | ((uint32_t)k << 4);
                        tc_mma(d_tmem, ad, bd, idesc, sfa_t, sfb_t, (uint32_t)((kb | k) != 0));
                    }
                    tc_commit(empty_bar(s));   // frees the smem stage once these MMAs have read it
                }
                if (ok) tc_commit(tfull_bar(as));
            }
            if (!ok) {
                // let MMAs already issued retire before TMEM is released
                tc_commit(drain_bar);
                uint64_t t0 = global_timer();
                while (!mbar_try_wait(drain_bar, 0) && global_timer() - t0 < WAIT_LIMIT_NS) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                 // TMEM lane quadrant this warp may read
        const int row_in_tile = q * 32 + lane;
        uint32_t acc_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++acc_it) {
            const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
            const int as = acc_it % C::ACC_STAGES;
            const uint32_t aph = (acc_it / C::ACC_STAGES) & 1u;
            ok = mbar_wait(tfull_bar(as), aph, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const int64_t row = (int64_t)tm * BM + row_in_tile;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + as * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tc_ld32(t_row + c * 32, v);
                tc_wait_ld();
                const int64_t col = (int64_t)tn * BN + c * 32;
                if (p.out_dtype == MXFP8_FP32) {
                    float4* d = reinterpret_cast<float4*>(static_cast<float*>(D) + row * p.N + col);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        d[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                           __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                } else {
                    uint4* d = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(D) + row * p.N + col);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t pk[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * j]),
                                                                           __uint_as_float(v[8 * i + 2 * j + 1]));
                            pk[j] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                        d[i] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(as));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// Byte matrix [outer, inner] row-major, box [box_outer, box_inner], 128-byte swizzle.
bool make_tmap(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint32_t box_inner, uint32_t box_outer)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {inner};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count()
{
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        return v;
    }();
    return n;
}

template <int BN>
int launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, const uint8_t* sfa, const uint8_t* sfb, void* D,
                GemmParams p, cudaStream_t stream)
{
    using C = Cfg<BN>;
    if (cudaFuncSetAttribute(gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_TOTAL) != cudaSuccess)
        return MXFP8_ERR_CUDA;
    p.tiles_m = (int)(p.M / BM);
    p.tiles_n = (int)(p.N / BN);
    p.num_tiles = p.tiles_m * p.tiles_n;
    p.num_kb = (int)(p.K / BK);
    const int sms = sm_count();
    if (sms <= 0) return MXFP8_ERR_CUDA;
    const int grid = p.num_tiles < sms ? p.num_tiles : sms;
    gemm_kernel<BN><<<grid, GEMM_THREADS, C::SMEM_TOTAL, stream>>>(ta, tb, sfa, sfb, D, p);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

}  // namespace
}  // namespace mxfp8

extern "C" size_t mxfp8_gemm_workspace_bytes(int64_t, int64_t, int64_t, int, int) { return 0; }

extern "C" int mxfp8_gemm(const void* Aq, const void* As, const void* Bq, const void* Bs,
                          int64_t M, int64_t N, int64_t K,
                          int a_major, int b_major, int a_elem, int b_elem,
                          void* D, int out_dtype, const mxfp8_epilogue* epi,
                          void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace mxfp8;
    (void)workspace; (void)workspace_bytes;
    if (a_major != MXFP8_K_MAJOR && a_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (b_major != MXFP8_K_MAJOR && b_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (a_elem != MXFP8_E4M3 && a_elem != MXFP8_E5M2) return MXFP8_ERR_ENUM;
    if (b_elem != MXFP8_E4M3 && b_elem != MXFP8_E5M2) return MXFP8_ERR_ENUM;
    if (out_dtype != MXFP8_FP32 && out_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (!Aq || !As || !Bq || !Bs) return MXFP8_ERR_NULL;
    if (!D && !epi) return MXFP8_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || (K % 32)) return MXFP8_ERR_SHAPE;
    if ((M % 128) || (N % 128) || (K % 128)) return MXFP8_ERR_UNSUPPORTED;
    if (M > 0x3FFFFFFF || N > 0x3FFFFFFF || K > 0x3FFFFFFF) return MXFP8_ERR_UNSUPPORTED;
    if (epi) return MXFP8_ERR_UNSUPPORTED;
    if (!aligned16(Aq) || !aligned16(As) || !aligned16(Bq) || !aligned16(Bs) || !aligned16(D)) return MXFP8_ERR_ALIGN;

    GemmParams p{};
    p.M = M; p.N = N; p.K = K;
    p.a_mn = a_major; p.b_mn = b_major; p.a_elem = a_elem; p.b_elem = b_elem; p.out_dtype = out_dtype;
    const bool wide = (N % 256) == 0;
    const uint32_t bn = wide ? 256 : 128;
    CUtensorMap ta, tb;
    const bool oka = a_major == MXFP8_K_MAJOR ? make_tmap(&ta, Aq, (uint64_t)K, (uint64_t)M, 128, 128)
                                              : make_tmap(&ta, Aq, (uint64_t)M, (uint64_t)K, 128, 128);
    const bool okb = b_major == MXFP8_K_MAJOR ? make_tmap(&tb, Bq, (uint64_t)K, (uint64_t)N, 128, bn)
                                              : make_tmap(&tb, Bq, (uint64_t)N, (uint64_t)K, 128, 128);
    if (!oka || !okb) return MXFP8_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint8_t* sa = static_cast<const uint8_t*>(As);
    const uint8_t* sb = static_cast<const uint8_t*>(Bs);
    return wide ? launch_gemm<256>(ta, tb, sa, sb, D, p, st) : launch_gemm<128>(ta, tb, sa, sb, D, p, st);
}
