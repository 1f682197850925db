// The TMA fast-path conversion kernels for the 6- and 4-bit element types of Table 1 (MXFP6: E2M3,
// E3M2; MXFP4: E2M1): the same kernels as for FP8 with another element type, compiled apart.
#include "quantize_tma_kernel.cuh"

namespace mxfp8 {

cudaError_t quantize_tma_launch_fp6_fp4(int elem, bool bf16_src, int orientation, bool emulate, const void* maps,
                                        const void* batch, cudaStream_t st)
{
    const QMaps& ms = *static_cast<const QMaps*>(maps);
    const QBatch& p = *static_cast<const QBatch*>(batch);
    switch (elem) {
        case MXFP8_E2M3: return quantize_tma_launch<MXFP8_E2M3>(bf16_src, orientation, emulate, ms, p, st);
        case MXFP8_E3M2: return quantize_tma_launch<MXFP8_E3M2>(bf16_src, orientation, emulate, ms, p, st);
        case MXFP8_E2M1: return quantize_tma_launch<MXFP8_E2M1>(bf16_src, orientation, emulate, ms, p, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace mxfp8
