// Host-side declarations shared by the translation units of the library (not public).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/mxfp8.h"

namespace mxfp8 {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// element types of the conversion kernels (Table 1) / of the tensor-core path of this library
inline bool valid_elem(int e) { return e == MXFP8_E4M3 || e == MXFP8_E5M2 || e == MXFP8_E2M3 || e == MXFP8_E3M2 || e == MXFP8_E2M1; }
inline bool fp8_elem(int e) { return e == MXFP8_E4M3 || e == MXFP8_E5M2; }

// Raises a kernel's dynamic shared-memory limit once per (kernel instantiation, device): the call
// costs several microseconds of host time and its effect lasts for the life of the context.
// `done` is a bit mask of devices, one static per call site.
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, unsigned long long& done)
{
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const unsigned long long bit = 1ull << (dev & 63);
    if (__atomic_load_n(&done, __ATOMIC_ACQUIRE) & bit) return cudaSuccess;
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (err == cudaSuccess) __atomic_fetch_or(&done, bit, __ATOMIC_RELEASE);
    return err;
}

// Launch accounting (mxfp8_launch_count).
int64_t launches();
void count_launch(int n);

// Device-pointer implementations behind the C entry points (arguments already validated).
int quantize_device(const void* src, int src_dtype, int64_t rows, int64_t cols, int orientation,
                    int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col,
                    int sf_layout, cudaStream_t stream);

// TMA fast path of mxfp8_quantize (quantize_tma.cu).
bool quantize_tma_eligible(int src_dtype, int64_t rows, int64_t cols);
int quantize_tma_device(const void* src, int src_dtype, int64_t rows, int64_t cols, int orientation,
                        int scale_rule, int elem, void* q_row, void* s_row, void* q_col, void* s_col,
                        int sf_layout, cudaStream_t stream, bool emulate = false);
// Several tensors of one dtype in one launch (same orientation, rule, element format, scale layout).
struct QuantizeItem {
    const void* src;
    int64_t rows, cols;
    void *q_row, *s_row, *q_col, *s_col;
};
int quantize_tma_batch(const QuantizeItem* items, int count, int src_dtype, int orientation, int scale_rule, int elem,
                       int sf_layout, cudaStream_t stream, bool emulate = false, int act = MXFP8_ACT_NONE,
                       const float* rstd = nullptr, const void* gamma = nullptr, bool gated = false,
                       const float* mean = nullptr, const void* beta = nullptr, const void* second_src = nullptr);
int quantize_read_and_clear_status();

// Device status word (bounded waits report here); defined in gemm.cu.
int read_and_clear_device_status(cudaStream_t stream);

}  // namespace mxfp8
