// Host side of the TMA fast path of mxfp8_quantize (kernels: quantize_tma_kernel.cuh) and the
// kernels of the two 8-bit element types; the 6- and 4-bit ones are compiled in quantize_tma_fp6_fp4.cu.
#include "quantize_tma_kernel.cuh"

namespace mxfp8 {

__device__ int g_quantize_status = 0;   // bounded TMA wait expired (read through mxfp8_device_status)
__device__ unsigned int g_quantize_sched[2 * StreamSlots::SLOTS];   // tile counters, two words per stream slot, zero between launches

int quantize_read_and_clear_status()
{
    int h = 0, z = 0;
    if (cudaMemcpyFromSymbol(&h, g_quantize_status, sizeof(int)) != cudaSuccess) return MXFP8_ERR_CUDA;
    if (h != 0 && cudaMemcpyToSymbol(g_quantize_status, &z, sizeof(int)) != cudaSuccess) return MXFP8_ERR_CUDA;
    return h == 0 ? MXFP8_OK : MXFP8_ERR_DEVICE_TIMEOUT;
}

// defined in quantize_tma_fp6_fp4.cu (opaque pointers: the batch types live in an unnamed namespace)
cudaError_t quantize_tma_launch_fp6_fp4(int elem, bool bf16_src, int orientation, bool emulate, const void* maps,
                                        const void* batch, cudaStream_t st);

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn qt_encode_fn()
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

bool make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, size_t esz, void* base, uint64_t cols, uint64_t rows,
                 uint32_t box_cols, uint32_t box_rows)
{
    EncodeTiledFn fn = qt_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * esz};
    const cuuint32_t box[2] = {box_cols, box_rows};
    static TensorMapCache<CUtensorMap> cache;
    const uint64_t kd[2] = {cols, rows}, ks[1] = {cols * esz};
    return cache.get(tensor_map_key(base, (uint32_t)dt, 2, kd, ks, box, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B), map,
                     [&](CUtensorMap* m) {
                         const cuuint32_t estr[2] = {1, 1};
                         return fn(m, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
                     });
}

}  // namespace

bool quantize_tma_eligible(int src_dtype, int64_t rows, int64_t cols)
{
    // TMA needs 16-byte row pitches for the source and for the byte outputs; tile counts must fit an int
    if (cols % 16) return false;
    const int64_t t_cols = (src_dtype == MXFP8_BF16) ? 128 : 64;
    const int64_t tiles = ((cols + t_cols - 1) / t_cols) * ((rows + T_ROWS - 1) / T_ROWS);
    return tiles < 0x7FFF0000LL && rows < 0x7FFFFFFFLL && cols < 0x7FFFFFFFLL && qt_encode_fn() != nullptr;
}

int quantize_tma_batch(const QuantizeItem* items, int count, int src_dtype, int orientation, int scale_rule, int elem,
                       int sf_layout, cudaStream_t stream, bool emulate, int act, const float* rstd, const void* gamma,
                       bool gated, const float* mean, const void* beta, const void* second_src)
{
    if (count < 1 || count > QT_MAX_TENSORS) return MXFP8_ERR_UNSUPPORTED;
    const bool bf = src_dtype == MXFP8_BF16;
    const uint32_t t_cols = bf ? 128 : 64;
    QMaps ms;
    QBatch p{};
    p.count = count;
    p.act = act;
    p.rstd = rstd;
    p.gamma = gamma;
    p.mean = mean;
    p.beta = beta;
    p.glu_cols = gated ? (int)items[0].cols : 0;     // gated: one tensor, source [rows, 2 * cols]
    p.up_map = second_src ? 1 : 0;                   // two sources of one shape: the second one rides in map 1
    int64_t tiles = 0;
    for (int i = 0; i < QT_MAX_TENSORS; ++i) {
        const QuantizeItem& it = items[i < count ? i : 0];
        if (i >= count && !(second_src && i == 1)) {   // unused slots repeat the first tensor's map: every map stays valid
            ms.m[i] = ms.m[0];
            continue;
        }
        if (second_src && i == 1) {
            if (count != 1 || gated) return MXFP8_ERR_UNSUPPORTED;
            if (!make_map_2d(&ms.m[1], bf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, bf ? 2 : 4,
                             const_cast<void*>(second_src), (uint64_t)it.cols, (uint64_t)it.rows, t_cols, T_ROWS))
                return MXFP8_ERR_CUDA;
            continue;
        }
        if (!make_map_2d(&ms.m[i], bf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, bf ? 2 : 4,
                         const_cast<void*>(it.src), (uint64_t)(gated ? 2 * it.cols : it.cols), (uint64_t)it.rows, t_cols, T_ROWS))
            return MXFP8_ERR_CUDA;
        if (i >= count) continue;
        QParams& q = p.t[i];
        q.rows = it.rows; q.cols = it.cols; q.rule = scale_rule; q.sf_layout = sf_layout;
        q.tiles_x = (int)((it.cols + t_cols - 1) / t_cols);
        q.tiles_x_magic = div_magic((uint32_t)q.tiles_x);
        q.tiles_y = (int)((it.rows + T_ROWS - 1) / T_ROWS);
        q.q_row = static_cast<uint8_t*>(it.q_row);
        q.q_col = static_cast<uint8_t*>(it.q_col);
        q.s_row = static_cast<uint8_t*>(it.s_row);
        q.s_col = static_cast<uint8_t*>(it.s_col);
        p.tile_start[i] = (int)tiles;
        tiles += (int64_t)q.tiles_x * q.tiles_y;
        if (tiles >= 0x7FFF0000LL) return MXFP8_ERR_UNSUPPORTED;   // the tile counter runs a few thousand past the last tile
    }
    for (int i = count; i <= QT_MAX_TENSORS; ++i) p.tile_start[i] = (int)tiles;
    // every device holds its own copy of the status word, at its own address
    static PerDeviceCache<int*> status_word;
    if (!status_word.get(p.status, [](int, int*& addr) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_quantize_status) != cudaSuccess) return false;
            addr = static_cast<int*>(ptr);
            return true;
        }))
        return MXFP8_ERR_CUDA;
    // the tile counter: two words per stream in a per-device array (kernels of one stream never overlap, so the words are
    // never shared); where no stream-owned words can be had (a launch being captured, too many streams) the kernel deals
    // tiles out by CTA index
    // (a launch of a few tiles per CTA has nothing to gain from it and keeps the runtime calls of the lookup off its host path)
    if (tiles > 4 * (int64_t)QT_CTAS_PER_SM * qt_sm_count()) {
        static StreamSlots slots;
        static PerDeviceCache<unsigned int*> sched_words;
        unsigned int* base = nullptr;
        const int slot = slots.get(stream);
        if (slot >= 0 && sched_words.get(base, [](int, unsigned int*& addr) {
                void* ptr = nullptr;
                if (cudaGetSymbolAddress(&ptr, g_quantize_sched) != cudaSuccess) return false;
                addr = static_cast<unsigned int*>(ptr);
                return true;
            }))
            p.sched = base + 2 * slot;
    }
#ifdef MXFP8_TEST_HOOKS
    if (const char* skip = getenv("MXFP8_TEST_SKIP_TILE")) p.test_skip_tile = atoi(skip);
#endif
    cudaError_t err;
    switch (elem) {
        case MXFP8_E4M3: err = quantize_tma_launch<MXFP8_E4M3>(bf, orientation, emulate, ms, p, stream); break;
        case MXFP8_E5M2: err = quantize_tma_launch<MXFP8_E5M2>(bf, orientation, emulate, ms, p, stream); break;
        default: err = quantize_tma_launch_fp6_fp4(elem, bf, orientation, emulate, &ms, &p, stream); break;
    }
    return err == cudaSuccess ? MXFP8_OK : MXFP8_ERR_CUDA;
}

}  // namespace mxfp8

namespace mxfp8 {
int quantize_tma_device(const void* src, int src_dtype, int64_t rows, int64_t cols, int orientation,
                        int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col,
                        int sf_layout, cudaStream_t stream, bool emulate)
{
    const QuantizeItem one{src, rows, cols, q_row, s_row, q_col, s_col};
    return quantize_tma_batch(&one, 1, src_dtype, orientation, scale_rule, elem, sf_layout, stream, emulate);
}
}  // namespace mxfp8
