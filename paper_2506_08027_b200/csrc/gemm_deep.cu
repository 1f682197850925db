// The DEEP variants of the GEMM kernel (reductions longer than one accumulation epoch), compiled apart from
// the others so that the two halves build side by side.
#include "gemm_kernel.cuh"

namespace mxfp8 {
namespace gemm {
#define MXFP8_GEMM_DEFINE_DEEP(BN, PAIR, MODE, EPI) \
    template int launch_kernel<BN, PAIR, MODE, EPI, true>(const GemmMaps&, const GemmParams&, int, cudaStream_t);
MXFP8_GEMM_VARIANTS(MXFP8_GEMM_DEFINE_DEEP)
#undef MXFP8_GEMM_DEFINE_DEEP
}  // namespace gemm
}  // namespace mxfp8
