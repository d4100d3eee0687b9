// placeholder until the chunked tensor-core kernel lands
#pragma once
#include <atomic>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "gf_wkv6.h"
namespace gf {
__device__ int g_dev_status = 0;
inline cudaError_t read_and_clear_device_status(int* flag)
{
    cudaError_t e = cudaMemcpyFromSymbol(flag, g_dev_status, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*flag) { int z = 0; e = cudaMemcpyToSymbol(g_dev_status, &z, sizeof(int)); }
    return e;
}
inline gf_status_t chunked_prefill(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
    const float*, const float*, float*, __nv_bfloat16*, const int32_t*, int, int, long long, int, cudaStream_t,
    std::atomic<uint64_t>*) { return GF_ERR_UNSUPPORTED; }
}
