// Measurement aid with no counterpart in the paper: the store-only and load-only HBM rates of the current
// device.  A copy moves one byte in for every byte out, so its rate says little about a kernel whose traffic is
// mostly stores (the fp32 output of the FC layers is 4 M N bytes against M K + N K bytes of Int8 operands);
// these two kernels give the one-directional ceilings that such a kernel runs against.
#include <cuda_runtime.h>
#include <stdint.h>

#include "q8_tools.h"

namespace q8 {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

// Every thread stores 16 bytes at a time, consecutive threads to consecutive addresses, grid-stride.
__global__ void __launch_bounds__(kThreads) hbm_store_kernel(uint4 *p, size_t n16, uint32_t tag)
{
    const size_t stride = (size_t)gridDim.x * kThreads;
    size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x;
    for (; i + (kUnroll - 1) * stride < n16; i += kUnroll * stride) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t v = tag ^ (uint32_t)(i + u * stride);
            __stcs(p + i + u * stride, make_uint4(v, v + 1u, v + 2u, v + 3u));
        }
    }
    for (; i < n16; i += stride) {
        const uint32_t v = tag ^ (uint32_t)i;
        __stcs(p + i, make_uint4(v, v + 1u, v + 2u, v + 3u));
    }
}

// Every thread loads 16 bytes at a time and folds them into a checksum that is stored only if it equals a
// value the caller picks (so the loads cannot be optimised away and nothing is written otherwise).
__global__ void __launch_bounds__(kThreads) hbm_load_kernel(const uint4 *p, size_t n16, uint32_t never, uint32_t *sink)
{
    const size_t stride = (size_t)gridDim.x * kThreads;
    size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x;
    uint32_t acc = 0;
    for (; i + (kUnroll - 1) * stride < n16; i += kUnroll * stride) {
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = __ldcs(p + i + u * stride);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) acc ^= v[u].x + v[u].y + v[u].z + v[u].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldcs(p + i);
        acc ^= v.x + v.y + v.z + v.w;
    }
    if (acc == never && sink != nullptr) *sink = acc;
}

}  // namespace
}  // namespace q8

extern "C" q8_status q8_measure_hbm_peak(void *buf, size_t bytes, int store, int repeats, double *gbs, double *elapsed_ms,
                                         void *stream)
{
    using namespace q8;
    if (buf == nullptr || gbs == nullptr) return Q8_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(buf) & 15u) != 0) return Q8_ERR_ALIGN;
    if (bytes < 16 || repeats < 1 || repeats > 1000) return Q8_ERR_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return Q8_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return Q8_ERR_CUDA;
    const size_t n16 = bytes / 16;
    size_t want = (n16 + kThreads - 1) / kThreads;
    const unsigned grid = (unsigned)(want < (size_t)sms * 8 ? want : (size_t)sms * 8);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess) return Q8_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) {
        cudaEventDestroy(e0);
        return Q8_ERR_CUDA;
    }
    auto launch = [&](int r) {
        if (store) hbm_store_kernel<<<grid, kThreads, 0, s>>>(static_cast<uint4 *>(buf), n16, 0x9e3779b9u * (uint32_t)(r + 1));
        else hbm_load_kernel<<<grid, kThreads, 0, s>>>(static_cast<const uint4 *>(buf), n16, 0x7f4a7c15u, nullptr);
    };
    launch(0);  // warm-up
    q8_status result = Q8_OK;
    float ms = 0.0f;
    if (cudaEventRecord(e0, s) != cudaSuccess) result = Q8_ERR_CUDA;
    for (int r = 0; r < repeats && result == Q8_OK; ++r) launch(r + 1);
    if (result == Q8_OK && (cudaGetLastError() != cudaSuccess || cudaEventRecord(e1, s) != cudaSuccess ||
                            cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess ||
                            !(ms > 0.0f)))
        result = Q8_ERR_CUDA;
    if (result == Q8_OK) {
        *gbs = (double)(n16 * 16) * (double)repeats / (ms * 1e-3) / 1e9;
        if (elapsed_ms) *elapsed_ms = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return result;
}
