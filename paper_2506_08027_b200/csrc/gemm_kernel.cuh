// mxfp8_gemm: block-scaled MXFP8 matrix product on the 5th-generation tensor cores
// (Sec. 2 and App. A.3: per 32-element block dot product of the FP8 elements, scaled by the
// two blocks' UE8M0 scales, accumulated in FP32).
//
// Structure (one persistent CTA per SM, 320 threads, warp-specialised):
//   warp 0      TMA producer: A/B tiles (128-byte swizzle) and 512-byte scale atoms -> smem ring
//   warp 1      MMA issuer (one thread): tcgen05.cp scales smem->TMEM, then
//               tcgen05.mma.kind::mxf8f6f4.block_scale over the K loop; owns TMEM alloc/dealloc
//   Two variants of one kernel template:
//     PAIR = true : clusters of two CTAs work on one 256 x 256 tile with cta_group::2 MMAs.  Each
//                   CTA loads its own 128 rows of A and its own 128-row half of B (no multicast),
//                   all loads complete on the leader CTA's mbarrier, the leader issues the MMAs
//                   for both, and each CTA drains its own 128 x 256 accumulator.  The tensor
//                   core then reads only 8 KB of shared memory per CTA per MMA.
//     PAIR = false: one CTA per 128 x BN tile (BN = 256 or 128) with cta_group::1, used when
//                   M is not a multiple of 256.
//   warps 2..9  epilogue: each warp drains its 32 lanes x BN/2 columns of the FP32 accumulator
//               into registers (tcgen05.ld), releases the accumulator at once so the next
//               tile's MMAs can start, then converts and writes D through a private 2 KB
//               64-byte-swizzled staging buffer with TMA stores
//   A CTA tile is 128 x BN (BN = 256 or 128) with K step 128 (= 4 MMAs of K = 32, one scale
//   byte per row per MMA = one 4-byte TMEM column entry per K step).
//   Every mbarrier wait is bounded: on expiry the kernel records MXFP8_ERR_DEVICE_TIMEOUT in
//   the device status word, raises an abort flag that all roles poll, drains and exits.
//   The same kernel runs, by template parameter MODE, one dense product, up to three independent
//   products as one pool of tiles (MULTI: mxfp8_gemm_multi), or the per-expert products of a
//   mixture-of-experts layer with the token axis split by device-side offsets (GROUP_M: tokens are
//   the rows of A; GROUP_K: tokens are the reduction axis): every role decodes "where does tile t
//   sit" through decode_tile() and shifts its TMA coordinates, K range and output rows accordingly.
//   Operands of any of the five element types of Table 1: the format codes go into the
//   instruction descriptor, 6- and 4-bit codes arrive in packed 16-byte slots.
#pragma once

#include <cuda.h>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mxfp8_device.cuh"
#include "mxfp8_host.h"

namespace mxfp8 {
namespace gemm {

constexpr int BM = 128;            // accumulator rows per CTA (TMEM lanes)
constexpr int BK = 128;            // K bytes per pipeline stage = one 128-byte swizzle row
constexpr int GEMM_THREADS = 320;
// The kernels run 384 threads in three warp groups: warps 0-3 (producer, MMA issuer, two idle warps) and the
// eight epilogue warps 4-11.  At launch each thread holds 168 registers (what twelve warps leave); the first group
// then shrinks to 104 registers per thread and the epilogue groups grow to 200 (setmaxnreg, placed at the top of each
// role's branch so that ptxas allocates every role against its own budget).  Why: the fused MXFP8 epilogue needs more
// than 168 registers -- with ten warps of 168 it spilled 40 per thread and the reloads missed the 30 KB of L1 that
// 223 KB of shared memory leave (600 000 local loads per launch, 4000 cycles per tile that nothing hid) -- and the
// plain kernels turned out 7-13 % faster per K block in this layout as well (8192^3: 638 -> 565 cycles per K block in
// an interleaved A/B run; the joint launch of the benchmark 0.485 -> 0.399 Mcycles).  The one exception found is the
// reduction-grouped WGRAD (tiles of 5-8 K blocks), 27 % slower in this layout: it keeps ten warps of 168 registers.
template <bool EPI, int MODE> struct Roles {
#ifdef MXFP8_GEMM_320
    static constexpr bool WIDE = EPI;
#else
    static constexpr bool WIDE = EPI || MODE != 2 /* GROUP_K */;
#endif
    static constexpr int THREADS = WIDE ? 384 : GEMM_THREADS;
    static constexpr int EPI_WARP0 = WIDE ? 4 : 2;      // first of the eight epilogue warps
    // 128 threads x 104 + 256 threads x 200 = 64 512 of the SM's 65 536 registers.  The split has to leave slack: the
    // launch allocates 168 per thread, the first group's decrease frees 128 x 64, the epilogue warps then ask for
    // 256 x 32, and a split that adds up to all 65 536 (112 / 200) left `setmaxnreg.inc` waiting for ever.
    static constexpr int REGS_FEW = 104, REGS_MANY = 200;
    static_assert(128 * REGS_FEW + 256 * REGS_MANY <= 65536 - 1024, "register split without slack");
};
constexpr int EPI_WARPS = 8;
constexpr int EPI_BUF_BYTES = 2048;   // 32 rows x 64 bytes per epilogue warp
constexpr int TMEM_COLS = 512;
#ifdef MXFP8_TEST_HOOKS
constexpr uint64_t WAIT_LIMIT_NS = 5000000ull;     // test build: bounded waits give up after 5 ms
#else
constexpr uint64_t WAIT_LIMIT_NS = 1000000000ull;  // bounded waits give up after 1 s
#endif
constexpr int KC_MAX_DEFAULT = 64;   // K blocks (of 128) that one accumulation epoch may span

// MULTI mode: several independent products share one launch (one pool of tiles over all of them)
constexpr int MAX_PROBLEMS = 3;
struct MultiProblem {
    int M, N;             // output extent
    int a_mn, b_mn, a_elem, b_elem;
    int tiles_m, tiles_n, num_kb;
    int tile_start;       // first tile of this problem in the launch-wide numbering
    uint32_t stage_tx;
    uint8_t* d;           // output of this problem when its rows can be stored straight from registers (see d_direct), else null
};
struct ProblemMaps { CUtensorMap a, b, sfa, sfb, d; };
struct MultiMaps { ProblemMaps p[MAX_PROBLEMS]; };

struct GemmParams {
    int64_t M, N, K;
    int a_mn, b_mn;       // 1 = MN-major storage
    int a_elem, b_elem;
    int out_dtype;
    int tiles_m, tiles_n, num_tiles, num_kb;
    int group_m;          // tile rasterisation: M-tiles per group (L2 reuse)
    uint32_t stage_tx;    // bytes that land per pipeline stage on the (leader's) full barrier
    int store_d;          // 0 when only the fused MXFP8 output is wanted
    int epi_orient;       // 0 = no fused MXFP8 output, else MXFP8_ROW / COL / BOTH
    int epi_rule, epi_elem;
    uint8_t* epi_q_row;   // fused MXFP8 bytes [M, N] of the two orientations (stored straight from the epilogue registers)
    uint8_t* epi_q_col;
    uint8_t* epi_s_row;   // swizzled scales of the row-blocked output, logical [M, N/32]
    uint8_t* epi_s_col;   // swizzled scales of the column-blocked output, logical [N, M/32]
    // grouped (per-expert) products: device array of num_groups + 1 token offsets, multiples of 128
    const int32_t* group_offsets;
    int num_groups;
    int token_limit;      // offsets may not pass this (tokens in the grouped tensor)
    int num_problems;     // MULTI
    MultiProblem mp[MAX_PROBLEMS];
    // Output rows stored straight from the epilogue registers (one 32-byte st.global.v8 per lane and 16 BF16 / 8 FP32
    // columns) instead of through the shared-memory staging buffer and a TMA store: the K loop of the 256 x 256 pair
    // tile keeps shared memory busy almost every cycle (33.5 KB of TMA writes + 32 KB of tensor-core reads per 512-cycle
    // K block at 128 B/clk), and the staged epilogue's 128 KB per tile came on top of that.  Needs a 32-byte aligned D
    // and a row pitch that is a multiple of 32 bytes; tiles that end beyond N, unaligned outputs and the adding
    // (SCATTER) mode keep the TMA path.  Null = TMA path only.
    uint8_t* d_direct;
    int kc_max;           // DEEP: longest run of K blocks accumulated inside the tensor core (see epoch_len)
    int test_skip_load;   // test builds only: 1 + index of the K block whose loads the producer leaves out (0 = none)
    int* status;          // device status word of this device (bounded waits and offset checks report here)
    unsigned long long* clock_probe;   // two words: SM cycles and nanoseconds that the first CTA was alive
    int rows_per_owner;   // SCATTER: D rows [r * rows_per_owner, (r + 1) * rows_per_owner) are added into owner r's buffer
    int tm_rot;           // SCATTER: M-tile this launch starts with (ranks start at different owners)
};

constexpr int MAX_GROUPS = 256;
// MODE of the kernel: one dense product, or one product per expert of a mixture-of-experts layer
//   GROUP_M: the rows of A (tokens) are grouped, B holds one matrix per expert   (fprop, dgrad)
//   GROUP_K: the reduction axis (tokens) is grouped, D holds one matrix per expert (wgrad)
//   MULTI  : up to MAX_PROBLEMS independent dense products, tiles of all of them dealt out as one pool
//   SCATTER: one dense product whose FP32 result is ADDED (TMA reduce) into per-owner buffers, row range by row
//            range; the buffers may be other GPUs' memory, so that the data-parallel sum of WGRAD partial
//            results and its scatter to the owners of the weight shards happen tile by tile inside the product
enum { DENSE = 0, GROUP_M = 1, GROUP_K = 2, MULTI = 3, SCATTER = 4 };
constexpr int MAX_OWNERS = 8;   // the owners' output maps take the place of MultiMaps (15 maps)
static_assert(sizeof(MultiMaps) >= MAX_OWNERS * sizeof(CUtensorMap), "owner maps must fit where the MULTI maps go");

// Modes whose 256-wide tiles use the two overlapping accumulators (see Cfg).  Measured in interleaved A/B runs, in
// cycles: single products -6 % at K = 2048 and at 8192^3 and nothing lost elsewhere, token-grouped products -2 %; but
// the joint launch of up to three products +14 % and the reduction-grouped WGRAD +36 %, so those (and the adding
// mode, not measured) keep the single accumulator.
__host__ __device__ constexpr bool overlap_for(int mode) { return mode == DENSE || mode == GROUP_M; }

// BN = accumulator columns per CTA = N extent of one tile (256, 192 or 128).  In PAIR mode a tile has 2*BM rows.
// BN = 192 and 128 have two accumulators side by side, so the epilogue of one tile runs under the MMAs of the next.
// Two 256-column accumulators plus scale columns do not fit into the 512 columns of TMEM, so at BN = 256 there is
// either one accumulator (OVL = false: every tile boundary waits for the whole drain) or two that OVERLAP (OVL = true):
// accumulator 0 at columns [0, 256), accumulator 1 at [224, 480); the 32 shared columns are the last 32 of a tile on
// accumulator 0 and the first 32 of a tile on accumulator 1.  The epilogue warps that own them drain them first and
// signal a barrier of their own (ovl); the next tile's MMAs wait for that barrier (and for the long-finished full drain
// of the tile before it).  The scales then alternate between two 12-column slots at [480, 504): tcgen05.cp and
// tcgen05.mma execute in issue order.  Which modes overlap is decided by measurement (overlap_for).
template <int BN, bool PAIR, bool OVL> struct Cfg {
    static constexpr bool OVERLAP = OVL && (BN == 256);
    static constexpr int ACC_STAGES = (BN == 256 && !OVERLAP) ? 1 : 2;
    static constexpr int ACC_STRIDE = OVERLAP ? BN - 32 : BN;
    static constexpr int B_ROWS = PAIR ? BN / 2 : BN;          // B rows (N indices) this CTA loads
    static constexpr int B_SLABS = (B_ROWS + 127) / 128;       // 128-wide slabs when B is MN-major
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES_K = B_ROWS * BK;              // bytes landing per stage, K-major B
    static constexpr int B_BYTES_MN = B_SLABS * 128 * BK;      // bytes landing per stage, MN-major B
    static constexpr int B_BYTES = B_BYTES_MN;                 // reservation (>= both)
    static constexpr int SFB_ATOMS = (BN + 127) / 128;         // a BN-wide tile starting at a multiple of 64 spans this many atoms
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + 512 + 512 * SFB_ATOMS;
    static constexpr int STAGES = (206 * 1024) / STAGE_BYTES > 8 ? 8 : (206 * 1024) / STAGE_BYTES;
    static constexpr int SF_COLS = 4 + 4 * SFB_ATOMS;          // TMEM columns of scales per stage
    static constexpr int SF_COL0 = ACC_STRIDE * (ACC_STAGES - 1) + BN;   // first scale column
    static constexpr int SMEM_A = 0;
    static constexpr int SMEM_B = SMEM_A + STAGES * A_BYTES;
    static constexpr int SMEM_SFA = SMEM_B + STAGES * B_BYTES;
    static constexpr int SMEM_SFB = SMEM_SFA + STAGES * 512;
    static constexpr int SMEM_EPI = SMEM_SFB + STAGES * 512 * SFB_ATOMS;      // 8 x 2 KB, 512-aligned
    static constexpr int NUM_BARS = 2 * STAGES + 2 * ACC_STAGES + 2;
    static constexpr int SMEM_BAR = SMEM_EPI + EPI_WARPS * EPI_BUF_BYTES;
    static constexpr int SMEM_MISC = SMEM_BAR + NUM_BARS * 8;  // tmem pointer, abort flag, bad-offsets flag
    static constexpr int SMEM_GROUPS = SMEM_MISC + 16;         // group offsets and first-tile indices, (MAX_GROUPS + 1) ints each
    static constexpr int SMEM_TOTAL = SMEM_GROUPS + 2 * (MAX_GROUPS + 1) * 4 + 4 + 1024;   // + slack to align the base to 1024
    static constexpr int SF_SLOTS = OVERLAP ? 2 : STAGES;      // scale slot of smem stage s: s % SF_SLOTS
    static_assert(SF_COL0 + SF_SLOTS * SF_COLS <= TMEM_COLS, "TMEM budget");
    static_assert(STAGES % SF_SLOTS == 0, "a stage keeps its scale slot from one pass over the ring to the next");
    static_assert(SMEM_TOTAL <= 227 * 1024, "shared memory budget");
    static_assert(SMEM_EPI % 512 == 0, "staging buffers need 512-byte alignment for the 64-byte swizzle");
    static_assert((BN / 2) % 32 == 0, "each epilogue warp owns whole 32-column chunks");
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
// arrive on a barrier addressed in the cluster's shared window (possibly the peer CTA's).  Default
// semantics (release at CTA scope): a cluster-scope release costs a memory fence of about a
// microsecond per tile, and nothing but the tcgen05-fenced TMEM hand-off is ordered by this barrier.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// cluster-window address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
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
// One lane of a converged warp, chosen by the hardware.  Code around it stays warp-uniform, so
// addresses and descriptors are computed once in the uniform datapath instead of per lane.
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xFFFFFFFF;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ uint64_t global_timer()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when the abort flag is up or the time limit passed (the latter also
// records the timeout and raises the flag for the other roles of this CTA).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status)
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
                atomicExch(status, (int)MXFP8_ERR_DEVICE_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
// Whole-warp wait of the two latency-critical roles (TMA producer, MMA issuer): all lanes spin
// on the non-blocking test so the warp reacts within a few cycles of the phase flip; the
// suspending try_wait costs a wake-up latency that the smem ring cannot hide.
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status)
{
    uint32_t spins = 0;
    uint64_t t0 = 0;
    bool ok = true;
    while (!mbar_test_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag) { ok = false; break; }
            const uint64_t now = global_timer();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                atomicExch(status, (int)MXFP8_ERR_DEVICE_TIMEOUT);
                ok = false;
                break;
            }
        }
    }
    return __all_sync(0xFFFFFFFFu, ok);
}
// TMA tile loads.  In PAIR mode the copy lands in this CTA's shared memory while the
// transaction bytes complete on the mbarrier address given (the leader CTA's barrier).
template <bool PAIR>
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1)
{
    if (PAIR)
        asm volatile(
            "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
            ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
    else
        asm volatile(
            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
            ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2)
{
    if (PAIR)
        asm volatile(
            "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
            ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
    else
        asm volatile(
            "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
            ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// arrive on `bar` (same offset in every CTA of the pair when PAIR) once all MMAs issued so far retire
template <bool PAIR>
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    if (PAIR)
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"((uint16_t)3) : "memory");
    else
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t desc)
{
    if (PAIR) asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
    else asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate)
{
    if (PAIR)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
            : "memory");
    else
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
__device__ __forceinline__ void tc_ld8(uint32_t taddr, uint32_t (&v)[8])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
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
__device__ __forceinline__ uint32_t make_idesc(int a_elem, int b_elem, int a_mn, int b_mn, int m, int n)
{
    return ((uint32_t)a_elem << 7) | ((uint32_t)b_elem << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------------ fused MXFP8 output
// 1/X exponent field for a block with this amax bit pattern (same integer form of Algorithm 1 /
// App. A.1 as the quantize kernels): e' = (bits + offset) >> 23, b = max(e' - emax, 0), field = 254 - b.
template <int ELEM>
__device__ __forceinline__ uint32_t epi_inv_exp(uint32_t amax_bits, uint32_t rule_offset)
{
    const int e = (int)((amax_bits + rule_offset) >> 23);
    return (uint32_t)min(254 + ElemTraits<ELEM>::emax - e, 254);
}
// This lane's 32 bytes of one output row, straight from registers to global memory: one 32-byte store where the
// address allows it, two 16-byte ones otherwise (the outputs are 16-byte aligned and N is a multiple of 128).
__device__ __forceinline__ void epi_store32(uint8_t* dst, const uint32_t (&w)[8])
{
    if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
    } else {
        asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
        asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 16), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
    }
}

// Converts this warp's 32 rows x CW columns of FP32 accumulators (lane = row) to MXFP8 exactly as
// mxfp8_quantize would convert the FP32 output (Sec. 2: the FP32 output is quantized to MX format
// when its consumer needs it): row blocks run along N inside a lane, column blocks are the warp's
// 32 rows (one warp-wide integer max per column; |x| bit patterns of finite floats order like integers).
//
// The work is a rolled loop over 32-column chunks: every pass converts the chunk held in v[0..31], stores its 32 bytes
// per row straight to global memory, and then moves the rest of the accumulator down by 32 registers (register files
// have no indexed access, so the data moves instead of the index).  One chunk's body is a tenth of the code that
// the straight-line form of both orientations over 128 columns took.  v is consumed.
template <int CW, int ELEM>
__device__ __forceinline__ void epi_mx(uint32_t (&v)[CW], const GemmParams& p, int lane, int row0, int col0)
{
    const uint32_t rule_offset = (p.epi_rule == MXFP8_RULE_PAPER) ? paper_offset<ELEM>() : 0u;
    const int row = row0 + lane;
    const bool do_row = (p.epi_orient & MXFP8_ROW) != 0, do_col = (p.epi_orient & MXFP8_COL) != 0;
    const int64_t nkb_col = p.M >> 5, kb_col = row0 >> 5;
    uint32_t srow = 0u;                   // this row's scale bytes of the warp's columns: adjacent bytes of one atom word
#pragma unroll 1
    for (int ch = 0; ch < CW / 32; ++ch) {
        const int c0 = col0 + ch * 32;
        if (do_row) {
            uint32_t wr[8];
            float m = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) m = fmaxf(m, fabsf(__uint_as_float(v[i])));   // NaN ignored
            if (m == INFINITY) {   // rare: finite-only maximum
                m = 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float a = fabsf(__uint_as_float(v[i]));
                    if (a < INFINITY) m = fmaxf(m, a);
                }
            }
            const uint32_t ie = epi_inv_exp<ELEM>(__float_as_uint(m), rule_offset);
            const float inv = __uint_as_float(ie << 23);
            srow |= (254u - ie) << (8 * ch);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                wr[i] = cvt_fp8x4<ELEM>(__uint_as_float(v[4 * i]) * inv, __uint_as_float(v[4 * i + 1]) * inv,
                                        __uint_as_float(v[4 * i + 2]) * inv, __uint_as_float(v[4 * i + 3]) * inv);
            epi_store32(p.epi_q_row + (int64_t)row * p.N + c0, wr);
        }
        if (do_col) {
            // Column c of the chunk is "owned" by lane c: one warp-wide integer max per column, the owner keeps the
            // result, derives scale and 1/X once, stores the scale byte, and hands 1/X out again by shuffle when the
            // column is cast.  Adding one exponent step makes the patterns of Inf and NaN wrap to negative numbers,
            // so a SIGNED max leaves them out of the maximum without a second pass.
            int own_biased = 0;
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                const int a = (int)((v[c] & 0x7FFFFFFFu) + 0x00800000u);
                int amax;
                asm volatile("redux.sync.max.s32 %0, %1, 0xffffffff;" : "=r"(amax) : "r"(a));
                if (lane == c) own_biased = amax;
            }
            const uint32_t own = (uint32_t)(max(own_biased, 0x00800000) - 0x00800000);   // no finite element: 0
            const uint32_t ie = epi_inv_exp<ELEM>(own, rule_offset);
            const float own_inv = __uint_as_float(ie << 23);
            uint32_t wc[8];
            p.epi_s_col[sf_swizzled_offset(c0 + lane, kb_col, nkb_col)] = (uint8_t)(254u - ie);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float y[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) y[e] = __uint_as_float(v[4 * i + e]) * __shfl_sync(0xFFFFFFFFu, own_inv, 4 * i + e);
                wc[i] = cvt_fp8x4<ELEM>(y[0], y[1], y[2], y[3]);
            }
            epi_store32(p.epi_q_col + (int64_t)row * p.N + c0, wc);
        }
        // the next chunk moves down into v[0..31]
#pragma unroll
        for (int i = 0; i + 32 < CW; ++i) v[i] = v[i + 32];
    }
    if (do_row) {
        // the scale bytes of 128 columns are the four bytes of one word of the atom (64 columns: half a word)
        uint8_t* dst = p.epi_s_row + sf_swizzled_offset(row, col0 >> 5, p.N >> 5);
        if (CW == 128) *reinterpret_cast<uint32_t*>(dst) = srow;
        else *reinterpret_cast<uint16_t*>(dst) = (uint16_t)srow;
    }
}

// Tile rasterisation: tiles are numbered group by group; a group is `group_m` M-tiles tall and
// spans all N-tiles, M fastest inside it, so the tiles in flight at one time share few distinct
// A row-blocks and B row-blocks and hit in L2.
__device__ __forceinline__ void tile_coords(int group_m, int tiles_m, int tiles_n, int tile, int& tm, int& tn)
{
    const int per_group = group_m * tiles_n;
    const int g = tile / per_group, r = tile - g * per_group;
    const int gm = min(group_m, tiles_m - g * group_m);
    tn = r / gm;
    tm = g * group_m + (r - tn * gm);
}

// Where one tile sits.  For a dense product everything but (tm, tn) is a constant; the grouped
// modes shift the operand coordinates to the tile's expert:
//   GROUP_M: A / SFA / D rows start at the expert's first token; B is the expert's matrix inside the
//            stack (K-major B [G*N, K]: N-coordinate + g*N; MN-major B [G*K, N]: K-coordinate + g*K)
//   GROUP_K: the K loop runs over the expert's tokens only; D rows start at g*M
struct TileCtx {
    int tm, tn;         // tile position inside its expert's output (rows in units of the tile height)
    int row0;           // added to A's MN coordinate (GROUP_M: the expert's first token)
    int d_row_extra;    // added on top of that for the D row (GROUP_K: g * M)
    int rows_end;       // D rows at or beyond this one are not stored
    int ka0, kb0;       // K-block offsets of A (and its scales) and of B (and its scales)
    int bn_off;         // added to B's MN coordinate
    int sfb_atom_off;   // added to the MN atom index of B's scales
    int nkb;            // K blocks of this tile
    int prob;           // MULTI: which product the tile belongs to
};

template <int MODE, int TM>
__device__ __forceinline__ TileCtx decode_tile(const GemmParams& p, const int* goff, const int* tstart, int tile, int& g)
{
    TileCtx t;
    t.prob = 0;
    if constexpr (MODE == MULTI) {
        while (g + 1 < p.num_problems && tile >= p.mp[g + 1].tile_start) ++g;      // tiles only move forward: g is a cursor
        const MultiProblem& q = p.mp[g];
        tile_coords(p.group_m, q.tiles_m, q.tiles_n, tile - q.tile_start, t.tm, t.tn);
        t.row0 = 0; t.d_row_extra = 0; t.rows_end = q.M; t.ka0 = 0; t.kb0 = 0; t.bn_off = 0; t.sfb_atom_off = 0;
        t.nkb = q.num_kb; t.prob = g;
    } else if constexpr (MODE == DENSE || MODE == SCATTER) {
        tile_coords(p.group_m, p.tiles_m, p.tiles_n, tile, t.tm, t.tn);
        if constexpr (MODE == SCATTER) { t.tm += p.tm_rot; if (t.tm >= p.tiles_m) t.tm -= p.tiles_m; }
        t.row0 = 0; t.d_row_extra = 0; t.rows_end = (int)p.M; t.ka0 = 0; t.kb0 = 0; t.bn_off = 0; t.sfb_atom_off = 0;
        t.nkb = p.num_kb;
    } else if constexpr (MODE == GROUP_M) {
        while (tile >= tstart[g + 1]) ++g;          // tiles only move forward: g is a cursor
        const int lo = goff[g], hi = goff[g + 1];
        tile_coords(p.group_m, (hi - lo + TM - 1) / TM, p.tiles_n, tile - tstart[g], t.tm, t.tn);
        t.row0 = lo; t.d_row_extra = 0; t.rows_end = hi; t.ka0 = 0; t.nkb = p.num_kb;
        if (p.b_mn) { t.kb0 = g * p.num_kb; t.bn_off = 0; t.sfb_atom_off = 0; }
        else { t.kb0 = 0; t.bn_off = g * (int)p.N; t.sfb_atom_off = (g * (int)p.N) >> 7; }
    } else {
        // experts are visited longest first (tstart[] holds that order here): the tiles that run side by side in
        // the persistent workers then have nearly the same K depth, and the short ones fill the end
        const int per_expert = p.tiles_m * p.tiles_n;
        const int slot = tile / per_expert;
        g = tstart[slot];
        tile_coords(p.group_m, p.tiles_m, p.tiles_n, tile - slot * per_expert, t.tm, t.tn);
        const int lo = goff[g], hi = goff[g + 1];
        t.row0 = 0; t.d_row_extra = g * (int)p.M; t.rows_end = (g + 1) * (int)p.M;
        t.ka0 = lo >> 7; t.kb0 = lo >> 7; t.bn_off = 0; t.sfb_atom_off = 0;
        t.nkb = (hi - lo) >> 7;
    }
    return t;
}

// K blocks this worker will run through: the flat loops of the producer and the MMA issuer count them.
template <int MODE>
__device__ __forceinline__ uint32_t worker_k_blocks(const GemmParams& p, const int* goff, const int* tstart, int num_tiles, int worker, int workers)
{
    if (num_tiles <= worker) return 0u;
    if constexpr (MODE == MULTI) {
        uint32_t total = 0;
        int g = 0;
        for (int tile = worker; tile < num_tiles; tile += workers) {
            while (g + 1 < p.num_problems && tile >= p.mp[g + 1].tile_start) ++g;
            total += (uint32_t)p.mp[g].num_kb;
        }
        return total;
    } else if constexpr (MODE != GROUP_K) {
        return (uint32_t)((num_tiles - worker + workers - 1) / workers) * (uint32_t)p.num_kb;
    } else {
        const int per_expert = p.tiles_m * p.tiles_n;
        uint32_t total = 0;
        for (int tile = worker; tile < num_tiles; tile += workers) {
            const int g = tstart[tile / per_expert];
            total += (uint32_t)((goff[g + 1] - goff[g]) >> 7);
        }
        return total;
    }
}

// Accumulation epochs (DEEP kernels).  The tensor core adds each 32-deep block dot product to its FP32
// accumulator by truncation, which biases long sums toward zero: measured relative Frobenius errors of
// 6.6e-6 at K = 16384 and 3.7e-5 at K = 65536 on gradient-like operands, against an acceptance bound of
// 1e-5.  Reductions deeper than kc_max K blocks are therefore cut into epochs of nearly equal length; each
// epoch starts a fresh accumulator, and the epilogue warps add the epochs' partial sums in registers with
// round-to-nearest FP32 additions (App. A.3: the block dot products are accumulated in FP32).  The MMA
// issuer and the epilogue warps both derive the epoch length from the tile's depth with this function.
__device__ __forceinline__ int epoch_len(int nkb, int kc_max)
{
    if (kc_max <= 0 || nkb <= kc_max) return nkb;
    const int n = (nkb + kc_max - 1) / kc_max;
    return (nkb + n - 1) / n;
}

// EPI: with the fused MXFP8 output compiled in (a separate instantiation: the plain kernels carry none of its code)
// DEEP: reductions longer than kc_max K blocks, summed in epochs (separate instantiations again, so that the
//       kernels of the common depths keep the straight-line epilogue)
template <int BN, bool PAIR, int MODE, bool EPI, bool DEEP>
__global__ void __launch_bounds__(Roles<EPI, MODE>::THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const __grid_constant__ CUtensorMap tmap_sfa, const __grid_constant__ CUtensorMap tmap_sfb,
            const __grid_constant__ CUtensorMap tmap_d, const __grid_constant__ CUtensorMap tmap_qrow,
            const __grid_constant__ CUtensorMap tmap_qcol, const __grid_constant__ MultiMaps mmaps,
            const __grid_constant__ GemmParams p)
{
    using C = Cfg<BN, PAIR, overlap_for(MODE)>;
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
    const uint32_t ovl_bar = drain_bar + 8u;   // OVERLAP: the columns that both accumulators use have been drained
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + C::SMEM_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::SMEM_MISC + 4);
    volatile int* bad_groups = reinterpret_cast<volatile int*>(base_ptr + C::SMEM_MISC + 8);
    int* goff = reinterpret_cast<int*>(base_ptr + C::SMEM_GROUPS);      // group offsets (tokens)
    int* tstart = goff + (MAX_GROUPS + 1);                              // GROUP_M: first tile of each group
    constexpr int TM = PAIR ? 2 * BM : BM;                              // tile height

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;   // 0 = leader (issues the MMAs)
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    const bool probe = blockIdx.x == 0 && threadIdx.x == 0;
    long long probe_c0 = 0;
    uint64_t probe_t0 = 0;
    if (probe) { probe_c0 = clock64(); probe_t0 = global_timer(); }
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < C::ACC_STAGES; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), (PAIR ? 2 : 1) * EPI_WARPS);
        }
        mbar_init(drain_bar, 1);
        mbar_init(ovl_bar, (PAIR ? 2 : 1) * (EPI_WARPS / 2));
        *abort_flag = 0;
        *bad_groups = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if constexpr (MODE == GROUP_M || MODE == GROUP_K) {
        // every CTA reads the offsets, checks them (non-negative, non-decreasing, multiples of 128,
        // inside the tensor) and, for GROUP_M, turns them into the first tile index of each group
        const int G = p.num_groups;
        for (int i = threadIdx.x; i <= G; i += Roles<EPI, MODE>::THREADS) goff[i] = p.group_offsets[i];
        __syncthreads();
        if (warp == 2) {
            bool bad = false;
            int run = 0;
            for (int i0 = 0; i0 < G; i0 += 32) {
                const int i = i0 + lane;
                int cnt = 0;
                if (i < G) {
                    const int lo = goff[i], hi = goff[i + 1];
                    if (lo < 0 || hi < lo || ((lo | hi) & 127) || hi > p.token_limit) bad = true;
                    else if (MODE == GROUP_M) cnt = ((hi - lo + TM - 1) / TM) * p.tiles_n;
                }
                int x = cnt;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
                    if (lane >= d) x += y;
                }
                if (MODE == GROUP_M && i < G) tstart[i + 1] = run + x;
                run += __shfl_sync(0xFFFFFFFFu, x, 31);
            }
            bad = __any_sync(0xFFFFFFFFu, bad);
            if (lane == 0) {
                if (MODE == GROUP_M) tstart[0] = 0;
                if (bad) { *bad_groups = 1; atomicExch(p.status, (int)MXFP8_ERR_DEVICE_ARGS); }
            }
        }
        if (MODE == GROUP_K && warp >= 2) {
            // tstart[k] = the expert with the k-th most tokens (ties by index): one thread per expert counts who comes before it
            const int i = (int)threadIdx.x - 64;
            if (i < G) {
                const int len = goff[i + 1] - goff[i];
                int rank = 0;
                for (int j = 0; j < G; ++j) {
                    const int other = goff[j + 1] - goff[j];
                    rank += (other > len || (other == len && j < i)) ? 1 : 0;
                }
                tstart[rank] = i;
            }
        }
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();      // the peer's barriers exist before anything remote touches them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // tiles of the whole launch (none when the offsets were rejected)
    const int num_tiles = (MODE == DENSE || MODE == MULTI || MODE == SCATTER) ? p.num_tiles
                        : (*bad_groups ? 0 : (MODE == GROUP_M ? tstart[p.num_groups] : p.num_groups * p.tiles_m * p.tiles_n));

    constexpr int EW0 = Roles<EPI, MODE>::EPI_WARP0;
    // EPI: the first warp group shrinks to REGS_FEW registers per thread, the epilogue warp groups grow to REGS_MANY
    if (warp == 0) {
        if constexpr (Roles<EPI, MODE>::WIDE) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Roles<EPI, MODE>::REGS_FEW));
        // ------------------------------------------------------------------ TMA producer
        // The whole warp walks the loop; one elected lane issues the copies.  Same flat,
        // ring-depth-unrolled loop as the MMA warp.
        {
            int a_mn = p.a_mn, b_mn = p.b_mn;
            uint32_t stage_tx = p.stage_tx;
            const CUtensorMap *ma = &tmap_a, *mb = &tmap_b, *msfa = &tmap_sfa, *msfb = &tmap_sfb;
            const uint32_t total = worker_k_blocks<MODE>(p, goff, tstart, num_tiles, worker, workers);
            int kb = 0, tile = worker, gcur = 0;
            int m_atom = 0, m0 = 0, n0 = 0, sfb_atom0 = 0, ka0 = 0, kb0 = 0, nkb = p.num_kb;
            uint32_t ph = 0;
            bool ok = true;
            for (uint32_t g0 = 0; g0 < total && ok; g0 += C::STAGES) {
#pragma unroll
                for (int s = 0; s < C::STAGES; ++s) {
                    if (g0 + s >= total) break;
                    if (kb == 0) {
                        TileCtx t = decode_tile<MODE, TM>(p, goff, tstart, tile, gcur);
                        if constexpr (MODE == GROUP_K) {
                            while (t.nkb == 0) { tile += workers; t = decode_tile<MODE, TM>(p, goff, tstart, tile, gcur); }   // expert without tokens
                        }
                        m0 = t.row0 + (t.tm * (PAIR ? 2 : 1) + (int)cta_rank) * BM;   // first row of A this CTA loads
                        m_atom = m0 >> 7;                                             // its scale atom
                        n0 = t.bn_off + t.tn * BN + (PAIR ? (int)cta_rank * C::B_ROWS : 0);    // first B row this CTA loads
                        sfb_atom0 = t.sfb_atom_off + ((t.tn * BN) >> 7);              // scale atom holding the tile's first column
                        ka0 = t.ka0; kb0 = t.kb0; nkb = t.nkb;
                        if constexpr (MODE == MULTI) {
                            const MultiProblem& q = p.mp[t.prob];
                            a_mn = q.a_mn; b_mn = q.b_mn; stage_tx = q.stage_tx;
                            ma = &mmaps.p[t.prob].a; mb = &mmaps.p[t.prob].b; msfa = &mmaps.p[t.prob].sfa; msfb = &mmaps.p[t.prob].sfb;
                        }
                    }
                    ok = warp_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status);
                    if (!ok) break;
                    // all bytes of the pair are counted on the leader's barrier
                    const uint32_t fb = PAIR ? map_to_cta(full_bar(s), 0) : full_bar(s);
                    const uint32_t sa = base + C::SMEM_A + s * C::A_BYTES;
                    const uint32_t sb = base + C::SMEM_B + s * C::B_BYTES;
                    const int k0a = (ka0 + kb) * BK, k0b = (kb0 + kb) * BK;
#ifdef MXFP8_TEST_HOOKS
                    // test builds: leave out the loads of one K block, so that the consumer's bounded wait runs out
                    // (nothing is in flight for that stage: the copies were never issued)
                    if (p.test_skip_load && g0 + s == (uint32_t)(p.test_skip_load - 1)) {
                        if (++kb == nkb) { kb = 0; tile += workers; }
                        continue;
                    }
#endif
                    if (elect_one()) {
                        if (cta_rank == 0) mbar_expect_tx(full_bar(s), stage_tx);
                        if (!a_mn) tma_load_2d<PAIR>(sa, ma, fb, k0a, m0);
                        else tma_load_2d<PAIR>(sa, ma, fb, m0, k0a);
                        if (!b_mn) {
                            tma_load_2d<PAIR>(sb, mb, fb, k0b, n0);
                        } else {
#pragma unroll
                            for (int j = 0; j < C::B_SLABS; ++j) tma_load_2d<PAIR>(sb + j * 16384, mb, fb, n0 + j * 128, k0b);
                        }
                        tma_load_3d<PAIR>(base + C::SMEM_SFA + s * 512, msfa, fb, 0, ka0 + kb, m_atom);
#pragma unroll
                        for (int j = 0; j < C::SFB_ATOMS; ++j)      // every CTA needs the scales of all BN columns
                            tma_load_3d<PAIR>(base + C::SMEM_SFB + (s * C::SFB_ATOMS + j) * 512, msfb, fb, 0, kb0 + kb,
                                              sfb_atom0 + j);
                    }
                    __syncwarp();
                    if (++kb == nkb) { kb = 0; tile += workers; }
                }
                ph ^= 1u;
            }
            if (!ok) {
                // give copies already in flight time to land before the CTA's smem is released
                for (int i = 0; i < 200; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        if constexpr (Roles<EPI, MODE>::WIDE) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Roles<EPI, MODE>::REGS_FEW));
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop so that descriptors stay in uniform registers; one
        // elected lane issues the tcgen05 instructions.  The loop runs over all K blocks of all
        // tiles of this worker and is unrolled by the ring depth, so the stage index is a
        // compile-time constant and every descriptor is "loop-invariant base + immediate".
        if (cta_rank == 0) {
            uint32_t idesc0 = make_idesc(p.a_elem, p.b_elem, p.a_mn, p.b_mn, PAIR ? 2 * BM : BM, BN);
            // Descriptors differ between stages and K steps only in the 14-bit start-address
            // field (16-byte units): keep the constant upper word and step the lower one.
            //   K-major : next K step = 32 bytes along the swizzled row (2 units); 8-row groups 1024 B apart.
            //   MN-major: next K step = 32 K-rows = 4096 bytes (256 units); 8-K-row groups 1024 B apart,
            //             128-wide MN slabs 16384 B apart.
            const uint32_t op_hi = (uint32_t)(smem_desc(0, 0, 1024, 2) >> 32);
            uint32_t a_lo0 = ((base + C::SMEM_A) >> 4) | (p.a_mn ? (16384u >> 4) << 16 : 0u);
            uint32_t b_lo0 = ((base + C::SMEM_B) >> 4) | (p.b_mn ? (16384u >> 4) << 16 : 0u);
            uint32_t a_kstep = p.a_mn ? 256u : 2u, b_kstep = p.b_mn ? 256u : 2u;
            const uint32_t sf_hi = (uint32_t)(smem_desc(0, 0, 128, 0) >> 32);   // scales: 32 rows x 16 B, 8-row groups 128 B apart
            const uint32_t sfa_lo0 = (base + C::SMEM_SFA) >> 4, sfb_lo0 = (base + C::SMEM_SFB) >> 4;
            auto desc64 = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | (uint64_t)lo; };
            const uint32_t total = worker_k_blocks<MODE>(p, goff, tstart, num_tiles, worker, workers);
            int kb = 0, tile = worker, gcur = 0, num_kb = p.num_kb;
            int kc = num_kb, ep_pos = 0;     // DEEP: epoch length of the tile, position inside the current epoch
            uint32_t ph = 0, acc_it = 0, d_tmem = tmem_base, sfb_skip = 0;
            int as = 0;
            bool ok = true;
            for (uint32_t g0 = 0; g0 < total && ok; g0 += C::STAGES) {
#pragma unroll
                for (int s = 0; s < C::STAGES; ++s) {
                    if (g0 + s >= total) break;
                    if (kb == 0) {   // first K block of a tile
                        // where the tile sits: worked out before the wait, so it runs under the epilogue's drain
                        TileCtx t = decode_tile<MODE, TM>(p, goff, tstart, tile, gcur);
                        if constexpr (MODE == GROUP_K) {
                            while (t.nkb == 0) { tile += workers; t = decode_tile<MODE, TM>(p, goff, tstart, tile, gcur); }   // expert without tokens
                        }
                        num_kb = t.nkb;
                        if constexpr (MODE == MULTI) {   // the product's own formats and majors
                            const MultiProblem& q = p.mp[t.prob];
                            idesc0 = make_idesc(q.a_elem, q.b_elem, q.a_mn, q.b_mn, PAIR ? 2 * BM : BM, BN);
                            a_lo0 = ((base + C::SMEM_A) >> 4) | (q.a_mn ? (16384u >> 4) << 16 : 0u);
                            b_lo0 = ((base + C::SMEM_B) >> 4) | (q.b_mn ? (16384u >> 4) << 16 : 0u);
                            a_kstep = q.a_mn ? 256u : 2u;
                            b_kstep = q.b_mn ? 256u : 2u;
                        }
                        // a tile that starts in the middle of a 128-wide scale atom reads its B scales from
                        // the matching TMEM column of the copied atoms (32 columns of B per TMEM column)
                        sfb_skip = (uint32_t)(((t.tn * BN) & 127) >> 5);
                        if constexpr (DEEP) {
                            kc = epoch_len(num_kb, p.kc_max);
                            ep_pos = 0;
                        } else {
                            // the accumulator must have been drained
                            as = acc_it % C::ACC_STAGES;
                            const uint32_t aph = (acc_it / C::ACC_STAGES) & 1u;
                            ok = warp_wait(tempty_bar(as), aph ^ 1u, abort_flag, p.status);
                            if (!ok) break;
                            if (C::OVERLAP && acc_it > 0) {   // the shared columns: drained by the accumulator use just before
                                ok = warp_wait(ovl_bar, (acc_it - 1u) & 1u, abort_flag, p.status);
                                if (!ok) break;
                            }
                            d_tmem = tmem_base + as * C::ACC_STRIDE;
                        }
                    }
                    if constexpr (DEEP) {
                        if (ep_pos == 0) {   // first K block of an epoch: the epoch's accumulator must have been drained
                            as = acc_it % C::ACC_STAGES;
                            const uint32_t aph = (acc_it / C::ACC_STAGES) & 1u;
                            ok = warp_wait(tempty_bar(as), aph ^ 1u, abort_flag, p.status);
                            if (!ok) break;
                            if (C::OVERLAP && acc_it > 0) {   // the shared columns: drained by the accumulator use just before
                                ok = warp_wait(ovl_bar, (acc_it - 1u) & 1u, abort_flag, p.status);
                                if (!ok) break;
                            }
                            d_tmem = tmem_base + as * C::ACC_STRIDE;
                        }
                    }
                    ok = warp_wait(full_bar(s), ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sfa_t = tmem_base + C::SF_COL0 + (s % C::SF_SLOTS) * C::SF_COLS;
                    const uint32_t sfb_t = sfa_t + 4;
                    if (elect_one()) {
                        tc_cp_sf<PAIR>(sfa_t, desc64(sfa_lo0 + s * (512 >> 4), sf_hi));
#pragma unroll
                        for (int j = 0; j < C::SFB_ATOMS; ++j)
                            tc_cp_sf<PAIR>(sfb_t + 4 * j, desc64(sfb_lo0 + (s * C::SFB_ATOMS + j) * (512 >> 4), sf_hi));
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint32_t idesc = idesc0 | ((uint32_t)k << 29) | ((uint32_t)k << 4);   // scale byte k of the column entry
                            tc_mma<PAIR>(d_tmem, desc64(a_lo0 + s * (C::A_BYTES >> 4) + k * a_kstep, op_hi),
                                         desc64(b_lo0 + s * (C::B_BYTES >> 4) + k * b_kstep, op_hi), idesc,
                                         sfa_t, sfb_t + sfb_skip, (uint32_t)(((DEEP ? ep_pos : kb) | k) != 0));
                        }
                        tc_commit<PAIR>(empty_bar(s));   // frees the smem stage (in both CTAs) once these MMAs have read it
                        if (kb == num_kb - 1 || (DEEP && ep_pos == kc - 1)) tc_commit<PAIR>(tfull_bar(as));
                    }
                    __syncwarp();
                    if constexpr (DEEP) {
                        ++kb;
                        if (++ep_pos == kc || kb == num_kb) { ep_pos = 0; ++acc_it; }
                        if (kb == num_kb) { kb = 0; tile += workers; }
                    } else {
                        if (++kb == num_kb) { kb = 0; tile += workers; ++acc_it; }
                    }
                }
                ph ^= 1u;
            }
            if (!ok) {
                // let MMAs already issued retire before TMEM is released
                if (elect_one()) tc_commit<PAIR>(drain_bar);
                __syncwarp();
                uint64_t t0 = global_timer();
                while (!mbar_try_wait(drain_bar, 0) && global_timer() - t0 < WAIT_LIMIT_NS) {}
            }
        }
    } else if (warp >= EW0) {
        if constexpr (Roles<EPI, MODE>::WIDE) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(Roles<EPI, MODE>::REGS_MANY));
        // ------------------------------------------------------------------ epilogue warps
        constexpr int CW = BN / 2;               // accumulator columns per epilogue warp
        const int q = warp & 3;                  // TMEM lane quadrant this warp may read
        const int half = (warp - EW0) >> 2;      // which half of the tile's columns
        const uint32_t buf = base + C::SMEM_EPI + (warp - EW0) * EPI_BUF_BYTES;
        // 64-byte swizzle of the staging buffer: 16-byte chunk j of row r sits at chunk j ^ ((r >> 1) & 3)
        const uint32_t row_off = buf + lane * 64;
        const uint32_t sw = (uint32_t)((lane >> 1) & 3);
        uint32_t acc_it = 0;
        bool ok = true;
        int n_total = (int)p.N;
        const CUtensorMap* md = &tmap_d;
        int gcur = 0;
        for (int tile = worker; tile < num_tiles && ok; tile += workers) {
            const TileCtx t = decode_tile<MODE, TM>(p, goff, tstart, tile, gcur);
            const int tm = t.tm, tn = t.tn;
            if constexpr (MODE == MULTI) { n_total = p.mp[t.prob].N; md = &mmaps.p[t.prob].d; }
            uint32_t v[CW];
            if (MODE == GROUP_K && t.nkb == 0) {
                // an expert without tokens: its product is all zeros and no MMA ran for this tile
#pragma unroll
                for (int c = 0; c < CW; ++c) v[c] = 0u;
            } else {
                const int as = acc_it % C::ACC_STAGES;
                const uint32_t aph = (acc_it / C::ACC_STAGES) & 1u;
                ++acc_it;
                if (lane == 0) ok = mbar_wait(tfull_bar(as), aph, abort_flag, p.status);   // one suspending poller per warp
                ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + as * C::ACC_STRIDE + half * CW;
                // OVERLAP: the warps of the upper half own the shared columns of a tile on accumulator 0 (its last chunk),
                // the warps of the lower half those of a tile on accumulator 1 (its first chunk): drained first, signalled at once
                const bool own_ovl = C::OVERLAP && half == (as ^ 1);
                const int ovl_c = as == 0 ? CW / 32 - 1 : 0;
                if (own_ovl) {
#pragma unroll
                    for (int c = 0; c < CW / 32; ++c)
                        if (c == ovl_c) tc_ld32(t_row + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[c * 32]));
                    tc_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (PAIR) mbar_arrive_cluster(map_to_cta(ovl_bar, 0));
                        else mbar_arrive(ovl_bar);
                    }
                }
#pragma unroll
                for (int c = 0; c < CW / 32; ++c)
                    if (!(own_ovl && c == ovl_c)) tc_ld32(t_row + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[c * 32]));
                tc_wait_ld();
                // the accumulator now lives in registers: hand TMEM back to the MMA warp of the leader
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(as), 0));
                    else mbar_arrive(tempty_bar(as));
                }
                if constexpr (DEEP) {
                    // the later epochs of a deep reduction: add their partial sums to the ones in registers
                    const int kc = epoch_len(t.nkb, p.kc_max);
                    for (int k0 = kc; k0 < t.nkb; k0 += kc) {
                        const int as2 = acc_it % C::ACC_STAGES;
                        const uint32_t aph2 = (acc_it / C::ACC_STAGES) & 1u;
                        ++acc_it;
                        if (lane == 0) ok = mbar_wait(tfull_bar(as2), aph2, abort_flag, p.status);
                        ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t t_row2 = tmem_base + ((uint32_t)(q * 32) << 16) + as2 * C::ACC_STRIDE + half * CW;
                        const bool own2 = C::OVERLAP && half == (as2 ^ 1);
                        const int ovl2 = as2 == 0 ? CW / 32 - 1 : 0;
#pragma unroll
                        for (int pass = 0; pass < 2; ++pass) {      // pass 0: the shared columns (their owner only), pass 1: the rest
#pragma unroll
                            for (int c = 0; c < CW / 8; ++c) {
                                if ((pass == 0) != (own2 && (c >> 2) == ovl2)) continue;
                                uint32_t w[8];
                                tc_ld8(t_row2 + c * 8, w);
                                tc_wait_ld();
#pragma unroll
                                for (int i = 0; i < 8; ++i)
                                    v[c * 8 + i] = __float_as_uint(__fadd_rn(__uint_as_float(v[c * 8 + i]), __uint_as_float(w[i])));
                            }
                            if (pass == 0 && own2) {
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) {
                                    if (PAIR) mbar_arrive_cluster(map_to_cta(ovl_bar, 0));
                                    else mbar_arrive(ovl_bar);
                                }
                            }
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(as2), 0));
                            else mbar_arrive(tempty_bar(as2));
                        }
                    }
                    if (!ok) break;
                }
            }

            int row0 = t.row0 + t.d_row_extra + (tm * (PAIR ? 2 : 1) + (int)cta_rank) * BM + q * 32;
            const int col0 = tn * BN + half * CW;
            const bool rows_inside = row0 < t.rows_end;      // ragged last M tile / rows of the next expert: a 32-row box entirely outside stores nothing
            if constexpr (MODE == SCATTER) {
                if (rows_inside) {   // this 32-row box lies inside one owner's row range (ranges are multiples of 128 rows)
                    const int owner = row0 / p.rows_per_owner;
                    md = reinterpret_cast<const CUtensorMap*>(&mmaps) + owner;
                    row0 -= owner * p.rows_per_owner;
                }
            }
            uint8_t* d_base = nullptr;
            if constexpr (MODE == MULTI) d_base = p.mp[t.prob].d;
            else if constexpr (MODE != SCATTER) d_base = p.d_direct;
            if (!p.store_d || !rows_inside) {
            } else if (MODE != SCATTER && d_base != nullptr && col0 + CW <= n_total) {
                // the whole column range of this warp lies inside the output: every lane stores its own row
                if (row0 + lane < t.rows_end) {
                    if (p.out_dtype == MXFP8_BF16) {
                        uint8_t* dst = d_base + ((int64_t)(row0 + lane) * n_total + col0) * 2;
#pragma unroll
                        for (int j = 0; j < CW / 16; ++j) {
                            uint32_t pk[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[j * 16 + 2 * e]),
                                                                                __uint_as_float(v[j * 16 + 2 * e + 1]));
                                pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
                            }
                            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                         ::"l"(dst + j * 32), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]),
                                           "r"(pk[6]), "r"(pk[7]) : "memory");
                        }
                    } else {
                        uint8_t* dst = d_base + ((int64_t)(row0 + lane) * n_total + col0) * 4;
#pragma unroll
                        for (int j = 0; j < CW / 8; ++j)
                            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                         ::"l"(dst + j * 32), "r"(v[j * 8]), "r"(v[j * 8 + 1]), "r"(v[j * 8 + 2]), "r"(v[j * 8 + 3]),
                                           "r"(v[j * 8 + 4]), "r"(v[j * 8 + 5]), "r"(v[j * 8 + 6]), "r"(v[j * 8 + 7]) : "memory");
                    }
                }
            } else if (p.out_dtype == MXFP8_BF16) {
#pragma unroll
                for (int ch = 0; ch < CW / 32; ++ch) {          // 32 columns = 64 bytes per row
                    if (col0 + ch * 32 >= n_total) break;       // ragged last tile: nothing to store
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t pk[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[ch * 32 + j * 8 + 2 * e]),
                                                                            __uint_as_float(v[ch * 32 + j * 8 + 2 * e + 1]));
                            pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
                        }
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(row_off + (((uint32_t)j ^ sw) << 4)), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(md), "r"(col0 + ch * 32), "r"(row0), "r"(buf) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            } else {
#pragma unroll
                for (int ch = 0; ch < CW / 16; ++ch) {          // 16 columns = 64 bytes per row
                    if (col0 + ch * 16 >= n_total) break;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(row_off + (((uint32_t)j ^ sw) << 4)), "r"(v[ch * 16 + j * 4]), "r"(v[ch * 16 + j * 4 + 1]),
                                       "r"(v[ch * 16 + j * 4 + 2]), "r"(v[ch * 16 + j * 4 + 3]) : "memory");
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        if constexpr (MODE == SCATTER)
                            asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(md), "r"(col0 + ch * 16), "r"(row0), "r"(buf) : "memory");
                        else
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(md), "r"(col0 + ch * 16), "r"(row0), "r"(buf) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
            // the fused MXFP8 output comes last: it consumes the accumulator registers
            if constexpr (EPI && CW % 64 == 0) {
                if (p.epi_orient && rows_inside && col0 < n_total) {   // N is a multiple of 128: a warp's columns are all inside or all outside
                    if (p.epi_elem == MXFP8_E4M3) epi_mx<CW, MXFP8_E4M3>(v, p, lane, row0, col0);
                    else epi_mx<CW, MXFP8_E5M2>(v, p, lane, row0, col0);
                }
            }
        }
        // all of this warp's stores must have left shared memory and reached global memory
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
    } else {
        if constexpr (Roles<EPI, MODE>::WIDE) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Roles<EPI, MODE>::REGS_FEW));   // the two idle warps of the first group
    }

    tc_fence_before();
    __syncthreads();
    if (probe) {
        p.clock_probe[0] = (unsigned long long)(clock64() - probe_c0);
        p.clock_probe[1] = (unsigned long long)(global_timer() - probe_t0);
    }
    if (PAIR) cluster_sync_all();      // nobody leaves while the peer may still signal this CTA's barriers
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

struct GemmMaps { CUtensorMap a, b, sfa, sfb, d, qrow, qcol; MultiMaps multi; };

// The launch itself; p is complete.  One instantiation per kernel variant; the DEEP ones are compiled in
// gemm_deep.cu (explicit instantiations), the others in gemm.cu.
template <int BN, bool PAIR, int MODE, bool EPI, bool DEEP>
int launch_kernel(const GemmMaps& m, const GemmParams& p, int workers, cudaStream_t stream)
{
    using C = Cfg<BN, PAIR, overlap_for(MODE)>;
    auto kernel = gemm_kernel<BN, PAIR, MODE, EPI, DEEP>;
    static unsigned long long smem_set = 0;
    if (ensure_dynamic_smem(kernel, C::SMEM_TOTAL, smem_set) != cudaSuccess) return MXFP8_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(PAIR ? 2 * workers : workers));
    cfg.blockDim = dim3(Roles<EPI, MODE>::THREADS);
    cfg.dynamicSmemBytes = C::SMEM_TOTAL;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, m.a, m.b, m.sfa, m.sfb, m.d, m.qrow, m.qcol, m.multi, p);
    if (getenv("MXFP8_LOG"))
        fprintf(stderr, "mxfp8_gemm launch grid=%u block=%d smem=%d tiles=%dx%d kblocks=%d%s -> %s\n", cfg.gridDim.x, Roles<EPI, MODE>::THREADS,
                C::SMEM_TOTAL, p.tiles_m, p.tiles_n, p.num_kb, DEEP ? " (epochs)" : "", cudaGetErrorString(err));
    count_launch(1);
    return err == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

// Per-device facts and addresses that the launches need (defined in gemm.cu).
struct GemmDevice {
    int sms;                           // multiprocessors
    int* status;                       // this device's copy of the status word
    unsigned long long* clock_probe;   // this device's copy of the clock probe
};
bool gemm_device(GemmDevice& out);

// Fills in what follows from the shape (tile counts, bytes per stage, epochs), picks the DEEP variant when a
// tile's reduction is longer than one epoch, sizes the grid and launches.
template <int BN, bool PAIR, int MODE = DENSE, bool EPI = false>
int launch_gemm(const GemmMaps& m, GemmParams p, cudaStream_t stream)
{
    using C = Cfg<BN, PAIR, overlap_for(MODE)>;
    p.tiles_m = (int)((p.M + (PAIR ? 2 * BM : BM) - 1) / (PAIR ? 2 * BM : BM));
    p.tiles_n = (int)((p.N + BN - 1) / BN);
    p.stage_tx = (PAIR ? 2u : 1u) * (uint32_t)(C::A_BYTES + (p.b_mn ? C::B_BYTES_MN : C::B_BYTES_K) + 512 + 512 * C::SFB_ATOMS);
    p.num_tiles = p.tiles_m * p.tiles_n;
    p.num_kb = (int)((p.K + BK - 1) / BK);   // a ragged K tail is zero-filled by TMA (operands) and by the scale pads
    p.group_m = 16;
    // MXFP8_GEMM_KC overrides the epoch length in K blocks (testing aid; 0 = never split a reduction)
    p.kc_max = KC_MAX_DEFAULT;
    if (const char* kc = getenv("MXFP8_GEMM_KC")) p.kc_max = atoi(kc);
    int deepest = p.num_kb;   // GROUP_K: an expert may hold all the tokens
    if (MODE == MULTI) {
        int64_t tiles = 0;
        deepest = 0;
        for (int i = 0; i < p.num_problems; ++i) {
            MultiProblem& q = p.mp[i];
            q.tiles_m = (q.M + (PAIR ? 2 * BM : BM) - 1) / (PAIR ? 2 * BM : BM);
            q.tiles_n = (q.N + BN - 1) / BN;
            q.stage_tx = (PAIR ? 2u : 1u) * (uint32_t)(C::A_BYTES + (q.b_mn ? C::B_BYTES_MN : C::B_BYTES_K) + 512 + 512 * C::SFB_ATOMS);
            q.tile_start = (int)tiles;
            tiles += (int64_t)q.tiles_m * q.tiles_n;
            if (tiles > 0x3FFFFFFF) return MXFP8_ERR_UNSUPPORTED;
            if (q.num_kb > deepest) deepest = q.num_kb;
        }
        p.num_tiles = (int)tiles;
    }
    GemmDevice dev;
    if (!gemm_device(dev)) return MXFP8_ERR_CUDA;
    p.status = dev.status;
    p.clock_probe = dev.clock_probe;
#ifdef MXFP8_TEST_HOOKS
    if (const char* skip = getenv("MXFP8_TEST_SKIP_LOAD")) p.test_skip_load = atoi(skip);
#endif
    const int max_workers = PAIR ? dev.sms / 2 : dev.sms;
    // tiles known to the host: all of them (dense), an upper bound (GROUP_M: every group may end in a
    // partly filled tile; the kernel counts the real ones), tiles of all experts (GROUP_K)
    int64_t host_tiles = p.num_tiles;
    if (MODE == GROUP_M) host_tiles = ((int64_t)p.tiles_m + p.num_groups) * p.tiles_n;
    if (MODE == GROUP_K) host_tiles = (int64_t)p.num_tiles * p.num_groups;
    const int workers = host_tiles < max_workers ? (int)host_tiles : max_workers;
    if (p.kc_max > 0 && deepest > p.kc_max) return launch_kernel<BN, PAIR, MODE, EPI, true>(m, p, workers, stream);
    return launch_kernel<BN, PAIR, MODE, EPI, false>(m, p, workers, stream);
}

// Every kernel variant that the entry points use
#define MXFP8_GEMM_VARIANTS(X)                                                                                       \
    X(256, true, DENSE, false) X(192, true, DENSE, false) X(256, false, DENSE, false) X(192, false, DENSE, false)    \
    X(128, false, DENSE, false) X(256, true, DENSE, true) X(256, false, DENSE, true) X(128, false, DENSE, true)      \
    X(256, true, GROUP_M, false) X(256, false, GROUP_M, false) X(256, true, GROUP_K, false) X(256, false, GROUP_K, false) \
    X(256, true, MULTI, false) X(256, true, SCATTER, false) X(192, true, SCATTER, false) X(128, false, SCATTER, false)
#define MXFP8_GEMM_DECLARE_DEEP(BN, PAIR, MODE, EPI) \
    extern template int launch_kernel<BN, PAIR, MODE, EPI, true>(const GemmMaps&, const GemmParams&, int, cudaStream_t);
MXFP8_GEMM_VARIANTS(MXFP8_GEMM_DECLARE_DEEP)
#undef MXFP8_GEMM_DECLARE_DEEP

}  // namespace gemm
}  // namespace mxfp8
