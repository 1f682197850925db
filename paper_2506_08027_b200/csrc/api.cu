// Host helpers of the C ABI: sizes, layout offsets, status strings, host-buffer variant.
#include "mxfp8_device.cuh"
#include <mutex>

#include "mxfp8_host.h"

extern "C" size_t mxfp8_scale_bytes(int64_t rows, int64_t cols, int orientation, int sf_layout)
{
    if (rows <= 0 || cols <= 0) return 0;
    if (orientation != MXFP8_ROW && orientation != MXFP8_COL) return 0;
    const int64_t mn = (orientation == MXFP8_ROW) ? rows : cols;
    const int64_t nkb = ((orientation == MXFP8_ROW) ? cols : rows) / 32;
    if (sf_layout == MXFP8_SF_LINEAR) return (size_t)(mn * nkb);
    if (sf_layout == MXFP8_SF_SWIZZLED) return (size_t)(((mn + 127) / 128) * ((nkb + 3) / 4) * 512);
    return 0;
}

extern "C" int64_t mxfp8_sf_offset(int64_t mn, int64_t kblock, int64_t n_kblocks, int sf_layout)
{
    if (mn < 0 || kblock < 0 || n_kblocks <= 0 || kblock >= n_kblocks) return -1;
    if (sf_layout == MXFP8_SF_LINEAR) return mn * n_kblocks + kblock;
    if (sf_layout == MXFP8_SF_SWIZZLED) return mxfp8::sf_swizzled_offset(mn, kblock, n_kblocks);
    return -1;
}

extern "C" const char* mxfp8_status_string(int status)
{
    switch (status) {
        case MXFP8_OK: return "ok";
        case MXFP8_ERR_NULL: return "null pointer";
        case MXFP8_ERR_ENUM: return "bad enum value";
        case MXFP8_ERR_SHAPE: return "bad shape (non-positive, or blocked dimension not a multiple of 32)";
        case MXFP8_ERR_ALIGN: return "misaligned pointer";
        case MXFP8_ERR_UNSUPPORTED: return "unsupported configuration";
        case MXFP8_ERR_CUDA: return "CUDA error";
        case MXFP8_ERR_DEVICE_TIMEOUT: return "bounded device wait expired";
        case MXFP8_ERR_WORKSPACE: return "workspace missing or too small";
        case MXFP8_ERR_DEVICE_ARGS: return "invalid values in a device-side argument array";
        default: return "unknown status";
    }
}

extern "C" int64_t mxfp8_launch_count(void) { return mxfp8::launches(); }

extern "C" int mxfp8_device_status(void* stream)
{
    return mxfp8::read_and_clear_device_status(static_cast<cudaStream_t>(stream));
}

namespace {
// One 16-byte piece per thread: atom (i, j) of part r goes to atom (i, r * atoms_part + j) of the whole.
__global__ void __launch_bounds__(256)
sf_concat_k_kernel(const uint4* __restrict__ parts, uint4* __restrict__ dst, int64_t atom_rows, int64_t atoms_part, int num_parts)
{
    const int64_t pieces = atom_rows * atoms_part * num_parts * 32;   // 32 pieces of 16 bytes per 512-byte atom
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < pieces; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t atom = t >> 5, piece = t & 31;
        const int64_t j = atom % atoms_part, ri = atom / atoms_part;   // destination order: (i, r, j)
        const int64_t r = ri % num_parts, i = ri / num_parts;
        dst[t] = parts[(((r * atom_rows + i) * atoms_part + j) << 5) + piece];
    }
}
}  // namespace

extern "C" int mxfp8_sf_concat_k(const void* parts, int num_parts, int64_t mn, int64_t k_part, void* dst, void* stream)
{
    if (!parts || !dst) return MXFP8_ERR_NULL;
    if (num_parts < 1 || mn <= 0 || k_part <= 0 || (k_part % 128)) return MXFP8_ERR_SHAPE;
    if (!mxfp8::aligned16(parts) || !mxfp8::aligned16(dst)) return MXFP8_ERR_ALIGN;
    const int64_t atom_rows = (mn + 127) / 128, atoms_part = k_part / 128;
    const int64_t pieces = atom_rows * atoms_part * num_parts * 32;
    const int64_t blocks = (pieces + 255) / 256;
    sf_concat_k_kernel<<<(unsigned)(blocks < 4096 ? blocks : 4096), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(parts), static_cast<uint4*>(dst), atom_rows, atoms_part, num_parts);
    mxfp8::count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

extern "C" int mxfp8_enable_peer_access(int peer_device)
{
    int dev = 0, can = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MXFP8_ERR_CUDA;
    if (peer_device == dev) return MXFP8_OK;
    if (cudaDeviceCanAccessPeer(&can, dev, peer_device) != cudaSuccess) { cudaGetLastError(); return MXFP8_ERR_SHAPE; }
    if (!can) return MXFP8_ERR_UNSUPPORTED;
    const cudaError_t err = cudaDeviceEnablePeerAccess(peer_device, 0);
    if (err == cudaErrorPeerAccessAlreadyEnabled) { cudaGetLastError(); return MXFP8_OK; }
    return err == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

namespace {
inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
}

extern "C" size_t mxfp8_quantize_host_ws_bytes(int src_dtype, int64_t rows, int64_t cols, int orientation)
{
    if (rows <= 0 || cols <= 0) return 0;
    const size_t esz = (src_dtype == MXFP8_BF16) ? 2 : 4;
    size_t total = up256((size_t)rows * cols * esz);
    for (int o = MXFP8_ROW; o <= MXFP8_COL; ++o)
        if (orientation & o) total += up256((size_t)rows * cols) + up256(mxfp8_scale_bytes(rows, cols, o, MXFP8_SF_SWIZZLED));
    return total;
}

extern "C" int mxfp8_quantize_host(const void* src_host, int src_dtype, int64_t rows, int64_t cols,
                                   int orientation, int scale_rule, int elem,
                                   void* q_row_host, void* s_row_host, void* q_col_host, void* s_col_host,
                                   int sf_layout, void* dev_ws, size_t dev_ws_bytes, void* stream)
{
    if (!src_host || !dev_ws) return MXFP8_ERR_NULL;
    if (src_dtype != MXFP8_FP32 && src_dtype != MXFP8_BF16) return MXFP8_ERR_ENUM;
    if (orientation < MXFP8_ROW || orientation > MXFP8_BOTH) return MXFP8_ERR_ENUM;
    if ((orientation & MXFP8_ROW) && (!q_row_host || !s_row_host)) return MXFP8_ERR_NULL;
    if ((orientation & MXFP8_COL) && (!q_col_host || !s_col_host)) return MXFP8_ERR_NULL;
    if (rows <= 0 || cols <= 0) return MXFP8_ERR_SHAPE;
    if (dev_ws_bytes < mxfp8_quantize_host_ws_bytes(src_dtype, rows, cols, orientation)) return MXFP8_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(dev_ws) & 255u) != 0) return MXFP8_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t esz = (src_dtype == MXFP8_BF16) ? 2 : 4;
    const size_t n = (size_t)rows * cols;
    char* p = static_cast<char*>(dev_ws);
    void* d_src = p; p += up256(n * esz);
    void *d_q[2] = {nullptr, nullptr}, *d_s[2] = {nullptr, nullptr};
    size_t s_bytes[2] = {0, 0};
    for (int o = 0; o < 2; ++o)
        if (orientation & (o + 1)) {
            s_bytes[o] = mxfp8_scale_bytes(rows, cols, o + 1, sf_layout);
            d_q[o] = p; p += up256(n);
            d_s[o] = p; p += up256(mxfp8_scale_bytes(rows, cols, o + 1, MXFP8_SF_SWIZZLED));
        }
    // whatever fails after the first copy has been queued: wait for the stream before the caller gets its buffers back
    auto fail = [&](int rc) { cudaStreamSynchronize(st); return rc; };
    if (cudaMemcpyAsync(d_src, src_host, n * esz, cudaMemcpyHostToDevice, st) != cudaSuccess) return fail(MXFP8_ERR_CUDA);
    const int rc = mxfp8_quantize(d_src, src_dtype, rows, cols, orientation, scale_rule, elem,
                                  d_q[0], d_s[0], d_q[1], d_s[1], sf_layout, stream);
    if (rc != MXFP8_OK) return fail(rc);
    void* h_q[2] = {q_row_host, q_col_host};
    void* h_s[2] = {s_row_host, s_col_host};
    for (int o = 0; o < 2; ++o)
        if (orientation & (o + 1)) {
            if (cudaMemcpyAsync(h_q[o], d_q[o], n, cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(MXFP8_ERR_CUDA);
            if (cudaMemcpyAsync(h_s[o], d_s[o], s_bytes[o], cudaMemcpyDeviceToHost, st) != cudaSuccess) return fail(MXFP8_ERR_CUDA);
        }
    return cudaStreamSynchronize(st) == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

namespace {
struct LinearWs {
    char* src[3];      // X, W, dY (bf16); host variant only
    char* q[3][2];     // row / col quantized copies
    char* s[3][2];     // row / col scales (swizzled)
    char* out[3];      // Y, dX, dW (bf16); host variant only
    size_t total;
};

// Carves the scratch of one linear-layer step out of `base` (null: sizes only).  `staging` adds
// device copies of the three inputs and the three outputs for the host-buffer variant.
LinearWs plan_linear(char* base, int64_t T, int64_t H, int64_t F, bool staging)
{
    const int64_t shp[3][2] = {{T, H}, {F, H}, {T, F}};
    const int64_t outs[3][2] = {{T, F}, {T, H}, {F, H}};
    LinearWs w{};
    size_t off = 0;
    auto take = [&](size_t n) { char* p = base ? base + off : nullptr; off += up256(n); return p; };
    for (int t = 0; t < 3; ++t) {
        if (staging) w.src[t] = take((size_t)shp[t][0] * shp[t][1] * 2);
        for (int o = 0; o < 2; ++o) {
            w.q[t][o] = take((size_t)shp[t][0] * shp[t][1]);
            w.s[t][o] = take(mxfp8_scale_bytes(shp[t][0], shp[t][1], o + 1, MXFP8_SF_SWIZZLED));
        }
    }
    if (staging)
        for (int t = 0; t < 3; ++t) w.out[t] = take((size_t)outs[t][0] * outs[t][1] * 2);
    w.total = off;
    return w;
}

// The two launches of one step on device buffers: the three BOTH-orientation conversions in one, then
// FPROP, DGRAD and WGRAD in one (Sec. 3.2).
int linear_device(const LinearWs& w, const void* x, const void* wt, const void* dy, int64_t T, int64_t H, int64_t F,
                  int scale_rule, void* y, void* dx, void* dw, void* stream)
{
    const int64_t shp[3][2] = {{T, H}, {F, H}, {T, F}};
    const void* src[3] = {x, wt, dy};
    mxfp8_quantize_item items[3];
    for (int t = 0; t < 3; ++t) items[t] = mxfp8_quantize_item{src[t], shp[t][0], shp[t][1], w.q[t][0], w.s[t][0], w.q[t][1], w.s[t][1]};
    {   // the three casts share one launch
        const int rc = mxfp8_quantize_multi(items, 3, MXFP8_BF16, MXFP8_BOTH, scale_rule, MXFP8_E4M3, MXFP8_SF_SWIZZLED, stream);
        if (rc != MXFP8_OK) return rc;
    }
    enum { X = 0, W = 1, DY = 2, R = 0, C = 1 };
    // FPROP, DGRAD, WGRAD are independent once the copies exist: one launch over the tiles of all three
    const mxfp8_gemm_problem gemms[3] = {
        {w.q[X][R], w.s[X][R], w.q[W][R], w.s[W][R], T, F, H, MXFP8_K_MAJOR, MXFP8_K_MAJOR, MXFP8_E4M3, MXFP8_E4M3, y},
        {w.q[DY][R], w.s[DY][R], w.q[W][C], w.s[W][C], T, H, F, MXFP8_K_MAJOR, MXFP8_MN_MAJOR, MXFP8_E4M3, MXFP8_E4M3, dx},
        {w.q[DY][C], w.s[DY][C], w.q[X][C], w.s[X][C], F, H, T, MXFP8_MN_MAJOR, MXFP8_MN_MAJOR, MXFP8_E4M3, MXFP8_E4M3, dw},
    };
    return mxfp8_gemm_multi(gemms, 3, MXFP8_BF16, stream);
}

int linear_check(int64_t T, int64_t H, int64_t F, int scale_rule)
{
    if (T <= 0 || H <= 0 || F <= 0) return MXFP8_ERR_SHAPE;
    if (scale_rule != MXFP8_RULE_PAPER && scale_rule != MXFP8_RULE_OCP) return MXFP8_ERR_ENUM;
    if ((T % 128) || (H % 128) || (F % 128)) return MXFP8_ERR_UNSUPPORTED;
    return MXFP8_OK;
}
}  // namespace

extern "C" size_t mxfp8_linear_ws_bytes(int64_t T, int64_t H, int64_t F)
{
    if (T <= 0 || H <= 0 || F <= 0) return 0;
    return plan_linear(nullptr, T, H, F, false).total;
}

extern "C" int mxfp8_linear(const void* x, const void* w, const void* dy,
                            int64_t T, int64_t H, int64_t F, int scale_rule,
                            void* y, void* dx, void* dw, void* ws, size_t ws_bytes, void* stream)
{
    if (!x || !w || !dy || !y || !dx || !dw || !ws) return MXFP8_ERR_NULL;
    if (const int rc = linear_check(T, H, F, scale_rule)) return rc;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MXFP8_ERR_ALIGN;
    if (ws_bytes < mxfp8_linear_ws_bytes(T, H, F)) return MXFP8_ERR_WORKSPACE;
    return linear_device(plan_linear(static_cast<char*>(ws), T, H, F, false), x, w, dy, T, H, F, scale_rule, y, dx, dw, stream);
}

extern "C" size_t mxfp8_linear_host_ws_bytes(int64_t T, int64_t H, int64_t F)
{
    if (T <= 0 || H <= 0 || F <= 0) return 0;
    return plan_linear(nullptr, T, H, F, true).total;
}

namespace {
// Two helper streams and the events that tie them to the caller's stream, one set per device, made on
// first use and kept for the life of the process: the host variant overlaps the upload of dY with the
// download of Y (PCIe carries both directions at once).
constexpr int HOST_CHUNKS = 4;   // row chunks of the token axis in the host-buffer step

struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, w_in = nullptr, out_done = nullptr, dw_ready = nullptr;
    cudaEvent_t x_in[HOST_CHUNKS] = {}, dy_in[HOST_CHUNKS] = {}, y_ready[HOST_CHUNKS] = {}, dx_ready[HOST_CHUNKS] = {};
    bool ok = false;
    std::mutex busy;   // one host-buffer step at a time per device: the events above are shared
};

HostPipe* host_pipe()
{
    static HostPipe pipes[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    HostPipe& p = pipes[dev];
    if (!p.ok) {
        bool good = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess;
        auto make = [&](cudaEvent_t* e) { good = good && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
        make(&p.start); make(&p.w_in); make(&p.out_done); make(&p.dw_ready);
        for (int c = 0; c < HOST_CHUNKS; ++c) { make(&p.x_in[c]); make(&p.dy_in[c]); make(&p.y_ready[c]); make(&p.dx_ready[c]); }
        if (!good) return nullptr;
        p.ok = true;
    }
    return &p;
}
}  // namespace

extern "C" int mxfp8_linear_host(const void* x_host, const void* w_host, const void* dy_host,
                                 int64_t T, int64_t H, int64_t F, int scale_rule,
                                 void* y_host, void* dx_host, void* dw_host,
                                 void* dev_ws, size_t dev_ws_bytes, void* stream)
{
    if (!x_host || !w_host || !dy_host || !y_host || !dx_host || !dw_host || !dev_ws) return MXFP8_ERR_NULL;
    if (const int rc = linear_check(T, H, F, scale_rule)) return rc;
    if ((reinterpret_cast<uintptr_t>(dev_ws) & 255u) != 0) return MXFP8_ERR_ALIGN;
    if (dev_ws_bytes < mxfp8_linear_host_ws_bytes(T, H, F)) return MXFP8_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    HostPipe* hp = host_pipe();
    if (!hp) return MXFP8_ERR_CUDA;
    std::lock_guard<std::mutex> one_at_a_time(hp->busy);
    const LinearWs w = plan_linear(static_cast<char*>(dev_ws), T, H, F, true);
    enum { X = 0, W = 1, DY = 2, R = 0, C = 1 };
    // The token axis goes through in row chunks (whole 128-row scale atoms each), so that PCIe carries both directions
    // for most of the call: FPROP of a chunk starts when its rows of X have arrived and its rows of Y leave at once,
    // while dY is still coming in; DGRAD likewise per chunk of dY.  Row-blocked copies are made per chunk, the
    // column-blocked ones (blocks run down the token axis) once per tensor when all of it is there.  Every product
    // is the same tile arithmetic as in mxfp8_linear, so the results are bit-identical.
    const int chunks = (T % (128 * HOST_CHUNKS) == 0) ? HOST_CHUNKS : 1;
    const int64_t Tc = T / chunks;
    const int64_t s_row_chunk_x = (Tc / 128) * ((H / 32 + 3) / 4) * 512;    // bytes of swizzled row scales per chunk of X
    const int64_t s_row_chunk_dy = (Tc / 128) * ((F / 32 + 3) / 4) * 512;   // ... and of dY
    const size_t wb = (size_t)F * H * 2;
    // A failure half way leaves copies to and from the caller's buffers queued on three streams: wait for them before
    // handing the buffers back with the error.
    auto fail = [&](int rc) {
        cudaStreamSynchronize(hp->in);
        cudaStreamSynchronize(st);
        cudaStreamSynchronize(hp->out);
        return rc;
    };
#define MXFP8_TRY(call) do { if ((call) != cudaSuccess) return fail(MXFP8_ERR_CUDA); } while (0)
#define MXFP8_RC(call) do { const int rc_ = (call); if (rc_ != MXFP8_OK) return fail(rc_); } while (0)
    // uploads on the helper stream, behind whatever the caller's stream holds: W, then X and dY chunk by chunk
    MXFP8_TRY(cudaEventRecord(hp->start, st));
    MXFP8_TRY(cudaStreamWaitEvent(hp->in, hp->start, 0));
    MXFP8_TRY(cudaStreamWaitEvent(hp->out, hp->start, 0));
    MXFP8_TRY(cudaMemcpyAsync(w.src[W], w_host, wb, cudaMemcpyHostToDevice, hp->in));
    MXFP8_TRY(cudaEventRecord(hp->w_in, hp->in));
    for (int c = 0; c < chunks; ++c) {
        const size_t off = (size_t)c * Tc * H * 2;
        MXFP8_TRY(cudaMemcpyAsync(w.src[X] + off, static_cast<const char*>(x_host) + off, (size_t)Tc * H * 2, cudaMemcpyHostToDevice, hp->in));
        MXFP8_TRY(cudaEventRecord(hp->x_in[c], hp->in));
    }
    for (int c = 0; c < chunks; ++c) {
        const size_t off = (size_t)c * Tc * F * 2;
        MXFP8_TRY(cudaMemcpyAsync(w.src[DY] + off, static_cast<const char*>(dy_host) + off, (size_t)Tc * F * 2, cudaMemcpyHostToDevice, hp->in));
        MXFP8_TRY(cudaEventRecord(hp->dy_in[c], hp->in));
    }
    // W: both orientations as soon as it is there
    MXFP8_TRY(cudaStreamWaitEvent(st, hp->w_in, 0));
    MXFP8_RC(mxfp8_quantize(w.src[W], MXFP8_BF16, F, H, MXFP8_BOTH, scale_rule, MXFP8_E4M3, w.q[W][R], w.s[W][R], w.q[W][C], w.s[W][C],
                            MXFP8_SF_SWIZZLED, stream));
    // FPROP chunk by chunk; Y rows leave on the second helper stream
    for (int c = 0; c < chunks; ++c) {
        const int64_t r0 = (int64_t)c * Tc;
        MXFP8_TRY(cudaStreamWaitEvent(st, hp->x_in[c], 0));
        MXFP8_RC(mxfp8_quantize(w.src[X] + r0 * H * 2, MXFP8_BF16, Tc, H, MXFP8_ROW, scale_rule, MXFP8_E4M3, w.q[X][R] + r0 * H,
                                w.s[X][R] + c * s_row_chunk_x, nullptr, nullptr, MXFP8_SF_SWIZZLED, stream));
        MXFP8_RC(mxfp8_gemm(w.q[X][R] + r0 * H, w.s[X][R] + c * s_row_chunk_x, w.q[W][R], w.s[W][R], Tc, F, H, MXFP8_K_MAJOR, MXFP8_K_MAJOR,
                            MXFP8_E4M3, MXFP8_E4M3, w.out[0] + r0 * F * 2, MXFP8_BF16, nullptr, nullptr, 0, stream));
        MXFP8_TRY(cudaEventRecord(hp->y_ready[c], st));
        MXFP8_TRY(cudaStreamWaitEvent(hp->out, hp->y_ready[c], 0));
        MXFP8_TRY(cudaMemcpyAsync(static_cast<char*>(y_host) + r0 * F * 2, w.out[0] + r0 * F * 2, (size_t)Tc * F * 2, cudaMemcpyDeviceToHost, hp->out));
    }
    // the column-blocked copy of X (for WGRAD) once all of X is there
    MXFP8_RC(mxfp8_quantize(w.src[X], MXFP8_BF16, T, H, MXFP8_COL, scale_rule, MXFP8_E4M3, nullptr, nullptr, w.q[X][C], w.s[X][C],
                            MXFP8_SF_SWIZZLED, stream));
    // DGRAD chunk by chunk as dY arrives
    for (int c = 0; c < chunks; ++c) {
        const int64_t r0 = (int64_t)c * Tc;
        MXFP8_TRY(cudaStreamWaitEvent(st, hp->dy_in[c], 0));
        MXFP8_RC(mxfp8_quantize(w.src[DY] + r0 * F * 2, MXFP8_BF16, Tc, F, MXFP8_ROW, scale_rule, MXFP8_E4M3, w.q[DY][R] + r0 * F,
                                w.s[DY][R] + c * s_row_chunk_dy, nullptr, nullptr, MXFP8_SF_SWIZZLED, stream));
        MXFP8_RC(mxfp8_gemm(w.q[DY][R] + r0 * F, w.s[DY][R] + c * s_row_chunk_dy, w.q[W][C], w.s[W][C], Tc, H, F, MXFP8_K_MAJOR, MXFP8_MN_MAJOR,
                            MXFP8_E4M3, MXFP8_E4M3, w.out[1] + r0 * H * 2, MXFP8_BF16, nullptr, nullptr, 0, stream));
        MXFP8_TRY(cudaEventRecord(hp->dx_ready[c], st));
        MXFP8_TRY(cudaStreamWaitEvent(hp->out, hp->dx_ready[c], 0));
        MXFP8_TRY(cudaMemcpyAsync(static_cast<char*>(dx_host) + r0 * H * 2, w.out[1] + r0 * H * 2, (size_t)Tc * H * 2, cudaMemcpyDeviceToHost, hp->out));
    }
    // WGRAD needs every token: column-blocked dY, then the product, then dW leaves
    MXFP8_RC(mxfp8_quantize(w.src[DY], MXFP8_BF16, T, F, MXFP8_COL, scale_rule, MXFP8_E4M3, nullptr, nullptr, w.q[DY][C], w.s[DY][C],
                            MXFP8_SF_SWIZZLED, stream));
    MXFP8_RC(mxfp8_gemm(w.q[DY][C], w.s[DY][C], w.q[X][C], w.s[X][C], F, H, T, MXFP8_MN_MAJOR, MXFP8_MN_MAJOR, MXFP8_E4M3, MXFP8_E4M3,
                        w.out[2], MXFP8_BF16, nullptr, nullptr, 0, stream));
    MXFP8_TRY(cudaEventRecord(hp->dw_ready, st));
    MXFP8_TRY(cudaStreamWaitEvent(hp->out, hp->dw_ready, 0));
    MXFP8_TRY(cudaMemcpyAsync(dw_host, w.out[2], wb, cudaMemcpyDeviceToHost, hp->out));
    MXFP8_TRY(cudaEventRecord(hp->out_done, hp->out));
    MXFP8_TRY(cudaStreamWaitEvent(st, hp->out_done, 0));
    MXFP8_TRY(cudaStreamSynchronize(st));
#undef MXFP8_TRY
#undef MXFP8_RC
    return mxfp8_device_status(stream);
}
