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
}
extern "C" size_t mxfp8_gemm_workspace_bytes(int64_t, int64_t, int64_t, int, int) { return 0; }
extern "C" int mxfp8_gemm(const void*, const void*, const void*, const void*, int64_t, int64_t, int64_t,
                          int, int, int, int, void*, int, const mxfp8_epilogue*, void*, size_t, void*)
{ return MXFP8_ERR_UNSUPPORTED; }
