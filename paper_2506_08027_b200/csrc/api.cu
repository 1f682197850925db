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
    if (cudaMemcpyAsync(d_src, src_host, n * esz, cudaMemcpyHostToDevice, st) != cudaSuccess) return MXFP8_ERR_CUDA;
    const int rc = mxfp8_quantize(d_src, src_dtype, rows, cols, orientation, scale_rule, elem,
                                  d_q[0], d_s[0], d_q[1], d_s[1], sf_layout, stream);
    if (rc != MXFP8_OK) return rc;
    void* h_q[2] = {q_row_host, q_col_host};
    void* h_s[2] = {s_row_host, s_col_host};
    for (int o = 0; o < 2; ++o)
        if (orientation & (o + 1)) {
            if (!h_q[o] || !h_s[o]) return MXFP8_ERR_NULL;
            if (cudaMemcpyAsync(h_q[o], d_q[o], n, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MXFP8_ERR_CUDA;
            if (cudaMemcpyAsync(h_s[o], d_s[o], s_bytes[o], cudaMemcpyDeviceToHost, st) != cudaSuccess) return MXFP8_ERR_CUDA;
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
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, xw_in = nullptr, dy_in = nullptr, y_ready = nullptr, y_out = nullptr;
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
        cudaEvent_t* evs[5] = {&p.start, &p.xw_in, &p.dy_in, &p.y_ready, &p.y_out};
        for (cudaEvent_t* e : evs) good = good && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
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
    const size_t xb = (size_t)T * H * 2, wb = (size_t)F * H * 2, yb = (size_t)T * F * 2;
#define MXFP8_TRY(call) do { if ((call) != cudaSuccess) return MXFP8_ERR_CUDA; } while (0)
#define MXFP8_RC(call) do { const int rc_ = (call); if (rc_ != MXFP8_OK) return rc_; } while (0)
    // uploads on the helper stream, behind whatever the caller's stream holds: X and W first, dY behind them
    MXFP8_TRY(cudaEventRecord(hp->start, st));
    MXFP8_TRY(cudaStreamWaitEvent(hp->in, hp->start, 0));
    MXFP8_TRY(cudaMemcpyAsync(w.src[W], w_host, wb, cudaMemcpyHostToDevice, hp->in));
    MXFP8_TRY(cudaMemcpyAsync(w.src[X], x_host, xb, cudaMemcpyHostToDevice, hp->in));
    MXFP8_TRY(cudaEventRecord(hp->xw_in, hp->in));
    MXFP8_TRY(cudaMemcpyAsync(w.src[DY], dy_host, yb, cudaMemcpyHostToDevice, hp->in));
    MXFP8_TRY(cudaEventRecord(hp->dy_in, hp->in));
    // FPROP as soon as X and W are on the device
    MXFP8_TRY(cudaStreamWaitEvent(st, hp->xw_in, 0));
    const mxfp8_quantize_item xw[2] = {
        {w.src[X], T, H, w.q[X][R], w.s[X][R], w.q[X][C], w.s[X][C]},
        {w.src[W], F, H, w.q[W][R], w.s[W][R], w.q[W][C], w.s[W][C]},
    };
    MXFP8_RC(mxfp8_quantize_multi(xw, 2, MXFP8_BF16, MXFP8_BOTH, scale_rule, MXFP8_E4M3, MXFP8_SF_SWIZZLED, stream));
    MXFP8_RC(mxfp8_gemm(w.q[X][R], w.s[X][R], w.q[W][R], w.s[W][R], T, F, H, MXFP8_K_MAJOR, MXFP8_K_MAJOR, MXFP8_E4M3,
                        MXFP8_E4M3, w.out[0], MXFP8_BF16, nullptr, nullptr, 0, stream));
    MXFP8_TRY(cudaEventRecord(hp->y_ready, st));
    // Y goes back on the second helper stream while dY is still coming in
    MXFP8_TRY(cudaStreamWaitEvent(hp->out, hp->y_ready, 0));
    MXFP8_TRY(cudaMemcpyAsync(y_host, w.out[0], yb, cudaMemcpyDeviceToHost, hp->out));
    MXFP8_TRY(cudaEventRecord(hp->y_out, hp->out));
    // DGRAD and WGRAD once dY has arrived
    MXFP8_TRY(cudaStreamWaitEvent(st, hp->dy_in, 0));
    MXFP8_RC(mxfp8_quantize(w.src[DY], MXFP8_BF16, T, F, MXFP8_BOTH, scale_rule, MXFP8_E4M3, w.q[DY][R], w.s[DY][R], w.q[DY][C],
                            w.s[DY][C], MXFP8_SF_SWIZZLED, stream));
    const mxfp8_gemm_problem grads[2] = {
        {w.q[DY][R], w.s[DY][R], w.q[W][C], w.s[W][C], T, H, F, MXFP8_K_MAJOR, MXFP8_MN_MAJOR, MXFP8_E4M3, MXFP8_E4M3, w.out[1]},
        {w.q[DY][C], w.s[DY][C], w.q[X][C], w.s[X][C], F, H, T, MXFP8_MN_MAJOR, MXFP8_MN_MAJOR, MXFP8_E4M3, MXFP8_E4M3, w.out[2]},
    };
    MXFP8_RC(mxfp8_gemm_multi(grads, 2, MXFP8_BF16, stream));
    MXFP8_TRY(cudaMemcpyAsync(dx_host, w.out[1], xb, cudaMemcpyDeviceToHost, st));
    MXFP8_TRY(cudaMemcpyAsync(dw_host, w.out[2], wb, cudaMemcpyDeviceToHost, st));
    MXFP8_TRY(cudaStreamWaitEvent(st, hp->y_out, 0));
    MXFP8_TRY(cudaStreamSynchronize(st));
#undef MXFP8_TRY
#undef MXFP8_RC
    return mxfp8_device_status(stream);
}
