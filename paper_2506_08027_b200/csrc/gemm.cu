// mxfp8_gemm and its relatives: entry points, tensor maps and tile choice.  The kernel is in gemm_kernel.cuh.
#include "gemm_kernel.cuh"

namespace mxfp8 {
using namespace gemm;

__device__ int g_device_status = 0;
// SM cycles and nanoseconds that the last GEMM launch's first CTA was alive: gives the SM clock the kernel really ran at
__device__ unsigned long long g_gemm_clock_probe[2] = {0ull, 0ull};

int read_and_clear_device_status(cudaStream_t stream)
{
    if (cudaStreamSynchronize(stream) != cudaSuccess) return MXFP8_ERR_CUDA;
    int h = 0, z = 0;
    if (cudaMemcpyFromSymbol(&h, g_device_status, sizeof(int)) != cudaSuccess) return MXFP8_ERR_CUDA;
    if (h != 0 && cudaMemcpyToSymbol(g_device_status, &z, sizeof(int)) != cudaSuccess) return MXFP8_ERR_CUDA;
    const int q = quantize_read_and_clear_status();
    if (q == MXFP8_ERR_CUDA) return q;
    if (h == MXFP8_ERR_DEVICE_ARGS) return h;
    return (h == 0 && q == MXFP8_OK) ? MXFP8_OK : MXFP8_ERR_DEVICE_TIMEOUT;
}

namespace {

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

// One cached encode call (see TensorMapCache).  strides: rank - 1 byte pitches.
bool encode_cached(CUtensorMap* map, CUtensorMapDataType dt, uint32_t rank, const void* base, const cuuint64_t* dims,
                   const cuuint64_t* strides, const cuuint32_t* box, CUtensorMapSwizzle swizzle, CUtensorMapL2promotion l2)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    static TensorMapCache<CUtensorMap> cache;
    uint64_t kd[3] = {0, 0, 0}, ks[2] = {0, 0};
    for (uint32_t i = 0; i < rank; ++i) kd[i] = dims[i];
    for (uint32_t i = 0; i + 1 < rank; ++i) ks[i] = strides[i];
    return cache.get(tensor_map_key(base, (uint32_t)dt, rank, kd, ks, box, (uint32_t)swizzle, (uint32_t)l2), map, [&](CUtensorMap* m) {
        const cuuint32_t estr[3] = {1, 1, 1};
        return fn(m, dt, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, l2,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Byte matrix [outer, inner] row-major, box [box_outer, box_inner], 128-byte swizzle.
bool make_tmap(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint32_t box_inner, uint32_t box_outer)
{
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {inner};
    const cuuint32_t box[2] = {box_inner, box_outer};
    return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Scale buffer in the 128x4 atom layout seen as [mn_atoms][k_atoms][128 x u32]; one box = one atom.
bool make_tmap_sf(CUtensorMap* map, const void* base, uint64_t mn_atoms, uint64_t k_atoms)
{
    const cuuint64_t dims[3] = {128, k_atoms, mn_atoms};
    const cuuint64_t strides[2] = {512, 512 * k_atoms};
    const cuuint32_t box[3] = {128, 1, 1};
    return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE,
                         CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// Fused MXFP8 output bytes [M, N]: boxes of 32 rows x 64 bytes, 64-byte swizzle (store side).
bool make_tmap_q(CUtensorMap* map, void* base, uint64_t M, uint64_t N)
{
    const cuuint64_t dims[2] = {N, M};
    const cuuint64_t strides[1] = {N};
    const cuuint32_t box[2] = {64u, 32u};
    return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B,
                         CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// Output matrix D [M, N] row-major: boxes of 32 rows x 64 bytes, 64-byte swizzle (store side).
bool make_tmap_d(CUtensorMap* map, void* base, uint64_t M, uint64_t N, int out_dtype)
{
    const bool f32 = out_dtype == MXFP8_FP32;
    const cuuint64_t dims[2] = {N, M};
    const cuuint64_t strides[1] = {N * (f32 ? 4u : 2u)};
    const cuuint32_t box[2] = {f32 ? 16u : 32u, 32u};
    return encode_cached(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box,
                         CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

}  // namespace
namespace gemm {
// Multiprocessor count and the addresses of this device's status word and clock probe, looked up once per device
// (every device that loads the library holds its own copy of the two symbols).
bool gemm_device(GemmDevice& out)
{
    static PerDeviceCache<GemmDevice> cache;
    return cache.get(out, [](int dev, GemmDevice& d) {
        void *s = nullptr, *c = nullptr;
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || d.sms <= 0) return false;
        if (cudaGetSymbolAddress(&s, g_device_status) != cudaSuccess || cudaGetSymbolAddress(&c, g_gemm_clock_probe) != cudaSuccess) return false;
        d.status = static_cast<int*>(s);
        d.clock_probe = static_cast<unsigned long long*>(c);
        return true;
    });
}
}  // namespace gemm
namespace {

// D can be stored straight from registers when every row segment of 32 bytes is aligned (see GemmParams::d_direct);
// MXFP8_GEMM_STAGED=1 forces the staged TMA path (testing aid)
uint8_t* direct_output(void* D, int64_t N, int out_dtype)
{
    const int64_t pitch = N * (out_dtype == MXFP8_FP32 ? 4 : 2);
    if (!D || (reinterpret_cast<uintptr_t>(D) & 31u) || (pitch & 31) || getenv("MXFP8_GEMM_STAGED")) return nullptr;
    return static_cast<uint8_t*>(D);
}

int sm_count()
{
    GemmDevice d;
    return gemm_device(d) ? d.sms : 0;
}

// Tile shape: estimated cycles = waves x (MMA cycles per tile + what the epilogue adds when it cannot run
// under the next tile's MMAs).  False when a forced shape (testing aid) does not apply to this problem.
bool choose_tile(int64_t M, int64_t N, int64_t K, bool epi, int sms, int& best_bn, bool& best_pair)
{
    best_bn = 128;
    best_pair = false;
    double best_cost = 1e300;
    // testing aid: MXFP8_GEMM_TILE = "256p" | "192p" | "256" | "192" | "128" forces a shape ("p" = CTA pair)
    const char* force = getenv("MXFP8_GEMM_TILE");
    for (int pass = force ? 0 : 1; pass < 2 && best_cost >= 1e300; ++pass)
    for (int bn : {256, 192, 128}) {
        for (int pr = 1; pr >= 0; --pr) {
            if (pr && (M <= 128 || bn == 128)) continue;
            if (epi && bn == 192) continue;   // the fused output works on 64-column chunks per epilogue warp
            if (pass == 0) {   // forced shape, when it applies to this problem
                if (atoi(force) != bn || (strchr(force, 'p') != nullptr) != (pr != 0)) continue;
            }
            const int64_t tiles = ((M + (pr ? 255 : 127)) / (pr ? 256 : 128)) * ((N + bn - 1) / bn);
            const int64_t workers = pr ? sms / 2 : sms;
            const int64_t waves = (tiles + workers - 1) / workers;
            // cycles per 128-deep K block measured on B200 for each shape (TMA feed and MMA issue
            // included), plus the part of the epilogue that cannot run under the next tile's MMAs
            const double kblock = pr ? (bn == 256 ? 624.0 : 747.0) : (bn == 256 ? 759.0 : (bn == 192 ? 770.0 : 450.0));
            const double per_tile = (double)(K / 128) * kblock + (bn == 256 ? 1600.0 : 300.0);
            const double cost = (double)waves * per_tile;
            if (cost < best_cost) { best_cost = cost; best_bn = bn; best_pair = pr != 0; }
        }
    }
    return best_cost < 1e300;
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
    using namespace mxfp8::gemm;
    (void)workspace; (void)workspace_bytes;
    if (a_major != MXFP8_K_MAJOR && a_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (b_major != MXFP8_K_MAJOR && b_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (!valid_elem(a_elem) || !valid_elem(b_elem)) return MXFP8_ERR_ENUM;
    if (out_dtype != MXFP8_FP32 && out_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (!Aq || !As || !Bq || !Bs) return MXFP8_ERR_NULL;
    if (!D && !epi) return MXFP8_ERR_NULL;
    if (epi) {
        if (epi->orientation < MXFP8_ROW || epi->orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
        if (epi->scale_rule != MXFP8_RULE_PAPER && epi->scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
        if (!valid_elem(epi->elem)) return MXFP8_ERR_ENUM;
        if (!fp8_elem(epi->elem)) return MXFP8_ERR_UNSUPPORTED;
        if ((epi->orientation & MXFP8_ROW) && (!epi->q_row || !epi->s_row)) return MXFP8_ERR_NULL;
        if ((epi->orientation & MXFP8_COL) && (!epi->q_col || !epi->s_col)) return MXFP8_ERR_NULL;
        if ((epi->orientation & MXFP8_ROW) && (!aligned16(epi->q_row) || !aligned16(epi->s_row))) return MXFP8_ERR_ALIGN;
        if ((epi->orientation & MXFP8_COL) && (!aligned16(epi->q_col) || !aligned16(epi->s_col))) return MXFP8_ERR_ALIGN;
    }
    if (M <= 0 || N <= 0 || K <= 0 || (K % 32)) return MXFP8_ERR_SHAPE;
    // TMA needs 16-byte row pitches: MN-major operands and the output constrain M and N
    if (a_major == MXFP8_MN_MAJOR && (M % 16)) return MXFP8_ERR_UNSUPPORTED;
    if (b_major == MXFP8_MN_MAJOR && (N % 16)) return MXFP8_ERR_UNSUPPORTED;
    if (D && (N % (out_dtype == MXFP8_FP32 ? 4 : 8))) return MXFP8_ERR_UNSUPPORTED;
    if (epi && ((M % 128) || (N % 128))) return MXFP8_ERR_UNSUPPORTED;   // the fused output writes whole scale atoms
    if (M > 0x3FFFFFFF || N > 0x3FFFFFFF || K > 0x3FFFFFFF) return MXFP8_ERR_UNSUPPORTED;
    if (!aligned16(Aq) || !aligned16(As) || !aligned16(Bq) || !aligned16(Bs) || (D && !aligned16(D))) return MXFP8_ERR_ALIGN;

    GemmParams p{};
    p.M = M; p.N = N; p.K = K;
    p.a_mn = a_major; p.b_mn = b_major; p.a_elem = a_elem; p.b_elem = b_elem; p.out_dtype = out_dtype;
    p.store_d = D ? 1 : 0;
    p.d_direct = direct_output(D, N, out_dtype);
    if (epi) {
        p.epi_orient = epi->orientation; p.epi_rule = epi->scale_rule; p.epi_elem = epi->elem;
        p.epi_q_row = static_cast<uint8_t*>(epi->q_row);
        p.epi_q_col = static_cast<uint8_t*>(epi->q_col);
        p.epi_s_row = static_cast<uint8_t*>(epi->s_row);
        p.epi_s_col = static_cast<uint8_t*>(epi->s_col);
    }
    const int sms = sm_count();
    if (sms <= 0) return MXFP8_ERR_CUDA;
    int best_bn = 128;
    bool best_pair = false;
    if (!choose_tile(M, N, K, epi != nullptr, sms, best_bn, best_pair)) return MXFP8_ERR_UNSUPPORTED;
    const uint32_t b_box_rows = (uint32_t)(best_pair ? best_bn / 2 : best_bn);   // K-major B rows per TMA box
    GemmMaps m;
    const bool oka = a_major == MXFP8_K_MAJOR ? make_tmap(&m.a, Aq, (uint64_t)K, (uint64_t)M, 128, 128)
                                              : make_tmap(&m.a, Aq, (uint64_t)M, (uint64_t)K, 128, 128);
    const bool okb = b_major == MXFP8_K_MAJOR ? make_tmap(&m.b, Bq, (uint64_t)K, (uint64_t)N, 128, b_box_rows)
                                              : make_tmap(&m.b, Bq, (uint64_t)N, (uint64_t)K, 128, 128);
    const bool oks = make_tmap_sf(&m.sfa, As, (uint64_t)((M + 127) / 128), (uint64_t)((K + 127) / 128)) &&
                     make_tmap_sf(&m.sfb, Bs, (uint64_t)((N + 127) / 128), (uint64_t)((K + 127) / 128));
    // maps that a launch does not use still have to be valid: point them at any output that exists
    void* q_any = epi ? ((epi->orientation & MXFP8_ROW) ? epi->q_row : epi->q_col) : D;
    const bool okd = D ? make_tmap_d(&m.d, D, (uint64_t)M, (uint64_t)N, out_dtype) : make_tmap_q(&m.d, q_any, (uint64_t)M, (uint64_t)N);
    const bool okq = true;
    if (okd) { m.qrow = m.d; m.qcol = m.d; }   // the fused output is stored from registers; these two only have to be valid maps
    if (getenv("MXFP8_LOG"))
        fprintf(stderr, "mxfp8_gemm M=%lld N=%lld K=%lld tile=%d%s maps: a=%d b=%d sf=%d d=%d q=%d\n", (long long)M, (long long)N,
                (long long)K, best_bn, best_pair ? "p" : "", (int)oka, (int)okb, (int)oks, (int)okd, (int)okq);
    if (!oka || !okb || !oks || !okd || !okq) return MXFP8_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (epi) {   // 192-wide tiles are never chosen with a fused output
        if (best_pair) return launch_gemm<256, true, DENSE, true>(m, p, st);
        return best_bn == 256 ? launch_gemm<256, false, DENSE, true>(m, p, st) : launch_gemm<128, false, DENSE, true>(m, p, st);
    }
    if (best_pair) return best_bn == 256 ? launch_gemm<256, true>(m, p, st) : launch_gemm<192, true>(m, p, st);
    if (best_bn == 256) return launch_gemm<256, false>(m, p, st);
    return best_bn == 192 ? launch_gemm<192, false>(m, p, st) : launch_gemm<128, false>(m, p, st);
}

extern "C" int mxfp8_grouped_gemm(const void* Aq, const void* As, const void* Bq, const void* Bs,
                                  const int32_t* group_offsets, int num_groups, int mode,
                                  int64_t M, int64_t N, int64_t K, int b_major, int a_elem, int b_elem,
                                  void* D, int out_dtype, void* stream)
{
    using namespace mxfp8;
    using namespace mxfp8::gemm;
    if (mode != MXFP8_GROUP_M && mode != MXFP8_GROUP_K) return MXFP8_ERR_ENUM;
    if (b_major != MXFP8_K_MAJOR && b_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (!valid_elem(a_elem) || !valid_elem(b_elem)) return MXFP8_ERR_ENUM;
    if (out_dtype != MXFP8_FP32 && out_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (!Aq || !As || !Bq || !Bs || !group_offsets || !D) return MXFP8_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || num_groups <= 0) return MXFP8_ERR_SHAPE;
    if (num_groups > MAX_GROUPS) return MXFP8_ERR_UNSUPPORTED;
    if (mode == MXFP8_GROUP_K && b_major != MXFP8_MN_MAJOR) return MXFP8_ERR_UNSUPPORTED;   // both operands are token-major
    // whole scale atoms per expert on every axis that is stacked or split
    if ((M % 128) || (N % 128) || (K % 128)) return MXFP8_ERR_UNSUPPORTED;
    const int64_t G = num_groups;
    const int64_t d_rows = mode == MXFP8_GROUP_M ? M : G * M;
    const int64_t b_stack = mode == MXFP8_GROUP_M ? (b_major == MXFP8_K_MAJOR ? G * N : G * K) : 0;
    if (M > 0x3FFFFFFF || N > 0x3FFFFFFF || K > 0x3FFFFFFF || d_rows > 0x3FFFFFFF || b_stack > 0x3FFFFFFF) return MXFP8_ERR_UNSUPPORTED;
    if (!aligned16(Aq) || !aligned16(As) || !aligned16(Bq) || !aligned16(Bs) || !aligned16(D) ||
        (reinterpret_cast<uintptr_t>(group_offsets) & 3u))
        return MXFP8_ERR_ALIGN;

    GemmParams p{};
    p.M = M; p.N = N; p.K = K;
    p.a_elem = a_elem; p.b_elem = b_elem; p.out_dtype = out_dtype;
    p.store_d = 1;
    // the reduction-grouped WGRAD (many short tiles, every one with a full output tile to write) is 15 % faster with the
    // staged TMA stores; the token-grouped products gain from the direct ones like the dense kernel
    p.d_direct = mode == MXFP8_GROUP_K ? nullptr : direct_output(D, N, out_dtype);
    p.group_offsets = group_offsets;
    p.num_groups = num_groups;
    const int sms = sm_count();
    if (sms <= 0) return MXFP8_ERR_CUDA;
    GemmMaps m;
    bool ok;
    bool pair;
    if (mode == MXFP8_GROUP_M) {
        // A [M tokens, K] K-major; B stacked per expert; D [M, N].  CTA pairs (256-row tiles) pay
        // off once an average expert fills a few of them; the host only knows the average.
        p.a_mn = 0; p.b_mn = b_major;
        p.token_limit = (int)M;
        pair = (M / G) >= 512;
        const char* force = getenv("MXFP8_GEMM_TILE");
        if (force) pair = strchr(force, 'p') != nullptr;
        ok = make_tmap(&m.a, Aq, (uint64_t)K, (uint64_t)M, 128, 128);
        ok = ok && (b_major == MXFP8_K_MAJOR ? make_tmap(&m.b, Bq, (uint64_t)K, (uint64_t)(G * N), 128, pair ? 128 : 256)
                                             : make_tmap(&m.b, Bq, (uint64_t)N, (uint64_t)(G * K), 128, 128));
        ok = ok && make_tmap_sf(&m.sfa, As, (uint64_t)(M / 128), (uint64_t)(K / 128));
        ok = ok && (b_major == MXFP8_K_MAJOR ? make_tmap_sf(&m.sfb, Bs, (uint64_t)(G * N / 128), (uint64_t)(K / 128))
                                             : make_tmap_sf(&m.sfb, Bs, (uint64_t)(N / 128), (uint64_t)(G * K / 128)));
        ok = ok && make_tmap_d(&m.d, D, (uint64_t)M, (uint64_t)N, out_dtype);
    } else {
        // A [K tokens, M] and B [K tokens, N], both MN-major with blocks down the token axis; D [G*M, N]
        p.a_mn = 1; p.b_mn = 1;
        p.token_limit = (int)K;
        pair = (M % 256) == 0;
        const char* force = getenv("MXFP8_GEMM_TILE");
        if (force) pair = strchr(force, 'p') != nullptr;
        ok = make_tmap(&m.a, Aq, (uint64_t)M, (uint64_t)K, 128, 128);
        ok = ok && make_tmap(&m.b, Bq, (uint64_t)N, (uint64_t)K, 128, 128);
        ok = ok && make_tmap_sf(&m.sfa, As, (uint64_t)(M / 128), (uint64_t)(K / 128));
        ok = ok && make_tmap_sf(&m.sfb, Bs, (uint64_t)(N / 128), (uint64_t)(K / 128));
        ok = ok && make_tmap_d(&m.d, D, (uint64_t)(G * M), (uint64_t)N, out_dtype);
    }
    if (getenv("MXFP8_LOG"))
        fprintf(stderr, "mxfp8_grouped_gemm mode=%d G=%d M=%lld N=%lld K=%lld tile=256%s maps=%d\n", mode, num_groups, (long long)M,
                (long long)N, (long long)K, pair ? "p" : "", (int)ok);
    if (!ok) return MXFP8_ERR_CUDA;
    m.qrow = m.d; m.qcol = m.d;   // no fused MXFP8 output in the grouped modes; the maps only have to be valid
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mode == MXFP8_GROUP_M) return pair ? launch_gemm<256, true, GROUP_M>(m, p, st) : launch_gemm<256, false, GROUP_M>(m, p, st);
    return pair ? launch_gemm<256, true, GROUP_K>(m, p, st) : launch_gemm<256, false, GROUP_K>(m, p, st);
}

extern "C" int mxfp8_gemm_multi(const mxfp8_gemm_problem* problems, int count, int out_dtype, void* stream)
{
    using namespace mxfp8;
    using namespace mxfp8::gemm;
    if (!problems) return MXFP8_ERR_NULL;
    if (count < 1) return MXFP8_ERR_SHAPE;
    if (count > MAX_PROBLEMS) return MXFP8_ERR_UNSUPPORTED;
    if (out_dtype != MXFP8_FP32 && out_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    GemmParams p{};
    p.out_dtype = out_dtype;
    p.store_d = 1;
    p.num_problems = count;
    GemmMaps m;
    // Deepest reductions first: the persistent workers take tiles round-robin in this order, so the launch ends on the
    // shallow tiles and the workers finish within one short tile of each other instead of one long one.
    int order[MAX_PROBLEMS] = {0, 1, 2};
    for (int i = 1; i < count; ++i)
        for (int j = i; j > 0 && problems[order[j]].K > problems[order[j - 1]].K; --j) { const int t = order[j]; order[j] = order[j - 1]; order[j - 1] = t; }
    for (int i = 0; i < MAX_PROBLEMS; ++i) {
        const mxfp8_gemm_problem& g = problems[i < count ? order[i] : order[0]];   // unused slots repeat the first product: every map stays valid
        if (i < count) {
            if (g.a_major != MXFP8_K_MAJOR && g.a_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
            if (g.b_major != MXFP8_K_MAJOR && g.b_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
            if (!valid_elem(g.a_elem) || !valid_elem(g.b_elem)) return MXFP8_ERR_ENUM;
            if (!g.Aq || !g.As || !g.Bq || !g.Bs || !g.D) return MXFP8_ERR_NULL;
            if (g.M <= 0 || g.N <= 0 || g.K <= 0 || (g.K % 32)) return MXFP8_ERR_SHAPE;
            if (g.a_major == MXFP8_MN_MAJOR && (g.M % 16)) return MXFP8_ERR_UNSUPPORTED;
            if (g.b_major == MXFP8_MN_MAJOR && (g.N % 16)) return MXFP8_ERR_UNSUPPORTED;
            if (g.N % (out_dtype == MXFP8_FP32 ? 4 : 8)) return MXFP8_ERR_UNSUPPORTED;
            if (g.M > 0x3FFFFFFF || g.N > 0x3FFFFFFF || g.K > 0x3FFFFFFF) return MXFP8_ERR_UNSUPPORTED;
            if (!aligned16(g.Aq) || !aligned16(g.As) || !aligned16(g.Bq) || !aligned16(g.Bs) || !aligned16(g.D)) return MXFP8_ERR_ALIGN;
            MultiProblem& q = p.mp[i];
            q.M = (int)g.M; q.N = (int)g.N; q.num_kb = (int)((g.K + BK - 1) / BK);
            q.d = direct_output(g.D, g.N, out_dtype);
            q.a_mn = g.a_major; q.b_mn = g.b_major; q.a_elem = g.a_elem; q.b_elem = g.b_elem;
        }
        ProblemMaps& pm = m.multi.p[i];
        if (i >= count) { pm = m.multi.p[0]; continue; }
        bool ok = g.a_major == MXFP8_K_MAJOR ? make_tmap(&pm.a, g.Aq, (uint64_t)g.K, (uint64_t)g.M, 128, 128)
                                             : make_tmap(&pm.a, g.Aq, (uint64_t)g.M, (uint64_t)g.K, 128, 128);
        ok = ok && (g.b_major == MXFP8_K_MAJOR ? make_tmap(&pm.b, g.Bq, (uint64_t)g.K, (uint64_t)g.N, 128, 128)   // pair tiles: 128 B rows per CTA
                                               : make_tmap(&pm.b, g.Bq, (uint64_t)g.N, (uint64_t)g.K, 128, 128));
        ok = ok && make_tmap_sf(&pm.sfa, g.As, (uint64_t)((g.M + 127) / 128), (uint64_t)((g.K + 127) / 128));
        ok = ok && make_tmap_sf(&pm.sfb, g.Bs, (uint64_t)((g.N + 127) / 128), (uint64_t)((g.K + 127) / 128));
        ok = ok && make_tmap_d(&pm.d, g.D, (uint64_t)g.M, (uint64_t)g.N, out_dtype);
        if (!ok) return MXFP8_ERR_CUDA;
    }
    // the single-product parameters and maps are unused in this mode but must be valid
    p.M = problems[order[0]].M; p.N = problems[order[0]].N; p.K = problems[order[0]].K;
    m.a = m.multi.p[0].a; m.b = m.multi.p[0].b; m.sfa = m.multi.p[0].sfa; m.sfb = m.multi.p[0].sfb; m.d = m.multi.p[0].d;
    m.qrow = m.d; m.qcol = m.d;
    return launch_gemm<256, true, MULTI>(m, p, static_cast<cudaStream_t>(stream));
}

extern "C" int mxfp8_gemm_reduce_scatter(const void* Aq, const void* As, const void* Bq, const void* Bs,
                                         int64_t M, int64_t N, int64_t K,
                                         int a_major, int b_major, int a_elem, int b_elem,
                                         void* const* D_owner, int num_owners, int first_owner, void* stream)
{
    using namespace mxfp8;
    using namespace mxfp8::gemm;
    if (a_major != MXFP8_K_MAJOR && a_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (b_major != MXFP8_K_MAJOR && b_major != MXFP8_MN_MAJOR) return MXFP8_ERR_ENUM;
    if (!valid_elem(a_elem) || !valid_elem(b_elem)) return MXFP8_ERR_ENUM;
    if (!Aq || !As || !Bq || !Bs || !D_owner) return MXFP8_ERR_NULL;
    if (num_owners < 1 || num_owners > MAX_OWNERS || first_owner < 0 || first_owner >= num_owners) return MXFP8_ERR_SHAPE;
    if (M <= 0 || N <= 0 || K <= 0 || (K % 32)) return MXFP8_ERR_SHAPE;
    if (M % ((int64_t)num_owners * 128)) return MXFP8_ERR_UNSUPPORTED;   // every owner holds whole 128-row tiles
    if (a_major == MXFP8_MN_MAJOR && (M % 16)) return MXFP8_ERR_UNSUPPORTED;
    if (b_major == MXFP8_MN_MAJOR && (N % 16)) return MXFP8_ERR_UNSUPPORTED;
    if (N % 4) return MXFP8_ERR_UNSUPPORTED;
    if (M > 0x3FFFFFFF || N > 0x3FFFFFFF || K > 0x3FFFFFFF) return MXFP8_ERR_UNSUPPORTED;
    if (!aligned16(Aq) || !aligned16(As) || !aligned16(Bq) || !aligned16(Bs)) return MXFP8_ERR_ALIGN;
    for (int r = 0; r < num_owners; ++r) {
        if (!D_owner[r]) return MXFP8_ERR_NULL;
        if (!aligned16(D_owner[r])) return MXFP8_ERR_ALIGN;
    }
    GemmParams p{};
    p.M = M; p.N = N; p.K = K;
    p.a_mn = a_major; p.b_mn = b_major; p.a_elem = a_elem; p.b_elem = b_elem; p.out_dtype = MXFP8_FP32;
    p.store_d = 1;
    p.rows_per_owner = (int)(M / num_owners);
    const int sms = sm_count();
    if (sms <= 0) return MXFP8_ERR_CUDA;
    int bn = 128;
    bool pair = false;
    if (!choose_tile(M, N, K, false, sms, bn, pair)) return MXFP8_ERR_UNSUPPORTED;
    if (!pair && bn != 128) { pair = M > 128; bn = pair ? bn : 128; }   // shapes built for this mode: 256p, 192p, 128
    // this launch begins with the tiles of owner `first_owner`, so that ranks do not all send to one GPU at a time
    p.tm_rot = (int)(((int64_t)first_owner * p.rows_per_owner) / (pair ? 2 * BM : BM));
    const uint32_t b_box_rows = (uint32_t)(pair ? bn / 2 : bn);
    GemmMaps m;
    bool ok = a_major == MXFP8_K_MAJOR ? make_tmap(&m.a, Aq, (uint64_t)K, (uint64_t)M, 128, 128)
                                       : make_tmap(&m.a, Aq, (uint64_t)M, (uint64_t)K, 128, 128);
    ok = ok && (b_major == MXFP8_K_MAJOR ? make_tmap(&m.b, Bq, (uint64_t)K, (uint64_t)N, 128, b_box_rows)
                                         : make_tmap(&m.b, Bq, (uint64_t)N, (uint64_t)K, 128, 128));
    ok = ok && make_tmap_sf(&m.sfa, As, (uint64_t)((M + 127) / 128), (uint64_t)((K + 127) / 128)) &&
         make_tmap_sf(&m.sfb, Bs, (uint64_t)((N + 127) / 128), (uint64_t)((K + 127) / 128));
    CUtensorMap* owner_maps = reinterpret_cast<CUtensorMap*>(&m.multi);
    for (int r = 0; r < num_owners && ok; ++r)
        ok = make_tmap_d(&owner_maps[r], D_owner[r], (uint64_t)p.rows_per_owner, (uint64_t)N, MXFP8_FP32);
    if (!ok) return MXFP8_ERR_CUDA;
    m.d = owner_maps[0]; m.qrow = m.d; m.qcol = m.d;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (pair) return bn == 256 ? launch_gemm<256, true, SCATTER>(m, p, st) : launch_gemm<192, true, SCATTER>(m, p, st);
    return launch_gemm<128, false, SCATTER>(m, p, st);
}

extern "C" int mxfp8_gemm_last_clock(void* stream, double* sm_mhz, double* kernel_us)
{
    if (!sm_mhz || !kernel_us) return MXFP8_ERR_NULL;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MXFP8_ERR_CUDA;
    unsigned long long h[2] = {0ull, 0ull};
    if (cudaMemcpyFromSymbol(h, mxfp8::g_gemm_clock_probe, sizeof(h)) != cudaSuccess) return MXFP8_ERR_CUDA;
    *kernel_us = (double)h[1] * 1e-3;
    *sm_mhz = h[1] ? (double)h[0] * 1e3 / (double)h[1] : 0.0;
    return MXFP8_OK;
}
