// Measurement aid with no counterpart in the paper: the rate at which the SMs of the current device can pull
// L2-resident operand tiles into shared memory with TMA, all SMs at once.  A 256 x 256 tile per SM pair makes the
// GEMM's main loop fetch 64 bytes per clock and SM at the full Int8 rate of the tensor cores, every byte of it from
// L2 (the operands of one FC layer fit there), so this rate tells whether L2 can feed the main loop when no operand
// byte is shared between SMs.  The kernel is the GEMM's producer side alone: `producers` warps (1 to 4) issue loads
// of 128-row x 128-byte boxes (the GEMM's operand box, 128-byte swizzle) into a ring of 12 stages, each warp into
// its own share of the stages, and as many warps hand the stages back as soon as their bytes have landed.
// Measured on a B200: one issuing warp manages a box per ~285 cycles (110 GB/s per SM, below the 64 B/clk the main
// loop wants: why the GEMM has two producer warps); two or more reach 214 GB/s per SM on all 148 SMs at once
// (31.7 TB/s, 112 B/clk) and 241 GB/s on one SM alone, so L2 is not what limits the main loop.  Every wait is bounded.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "q8_gemm_common.cuh"
#include "q8_internal.cuh"
#include "q8_sm100_ptx.cuh"
#include "q8_tools.h"

namespace q8 {
namespace {

using namespace ptx;
using namespace gemm_detail;

constexpr int kBoxRows = 128;
constexpr int kBoxBytes = kBoxRows * BLOCK_K;  // 16 KB
constexpr int kRing = 12;                      // 192 KB in flight per SM
constexpr int kMaxProducers = 4;
constexpr int kThreadsL2 = 2 * kMaxProducers * 32;
constexpr int kSmem = 1024 + kRing * kBoxBytes + 2 * kRing * 8 + 16;

__global__ void __launch_bounds__(kThreadsL2, 1)
l2_operand_kernel(const __grid_constant__ CUtensorMap tmap, int64_t boxes_k, int64_t num_boxes, int iters, int producers,
                  int32_t *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + kRing * kBoxBytes);
    uint64_t *empty_bar = full_bar + kRing;
    int *abort_flag = reinterpret_cast<int *>(empty_bar + kRing);
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // SM i walks the boxes i * iters, i * iters + 1, ... (mod the number of boxes): neighbours along K first, like
    // the k-blocks of a tile, and different SMs in different places of the matrix.  Warp w of the producers takes
    // the steps w, w + producers, ... and the stages w, w + producers, ... (producers divides the ring).
    const int per = kRing / producers;  // stages per producer
    if (warp < producers) {
        const uint32_t elected = elect_one();
        const int64_t first = ((int64_t)blockIdx.x * iters + warp) % num_boxes;
        int32_t kb = (int32_t)(first % boxes_k), rb = (int32_t)(first / boxes_k);
        const int32_t row_blocks = (int32_t)(num_boxes / boxes_k);
        int j = 0, issued = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int it = warp; it < iters; it += producers) {
            const int s = warp + j * producers;
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(empty_bar + s), phase ^ 1u, abort_flag, status));
            if (!ok) break;
            const uint32_t fb = smem_u32(full_bar + s);
            mbar_expect_tx_elected(elected, fb, kBoxBytes);
            tma_load_2d_elected(elected, smem_u32(smem + s * kBoxBytes), &tmap, kb * BLOCK_K, rb * kBoxRows, fb);
            ++issued;
            kb += producers;
            while (kb >= boxes_k) {
                kb -= (int32_t)boxes_k;
                if (++rb == row_blocks) rb = 0;
            }
            if (++j == per) { j = 0; phase ^= 1u; }
        }
        if (!ok) {
            // aborting: let this warp's copies already issued land before the CTA gives up its shared memory
            const uint64_t t0 = global_timer_ns();
            const int pending = issued < per ? issued : per;
            for (int i = 0; i < pending; ++i) {
                const int k = issued - 1 - i;  // the i-th most recent step of this warp
                const uint32_t par = (uint32_t)((k / per) & 1);
                while (!mbar_try_wait(smem_u32(full_bar + warp + (k % per) * producers), par) &&
                       global_timer_ns() - t0 < 50000000ull) {}
            }
        }
    } else if (warp >= kMaxProducers && warp < kMaxProducers + producers) {
        const int w = warp - kMaxProducers;
        int j = 0;
        uint32_t phase = 0;
        for (int it = w; it < iters; it += producers) {
            const int s = w + j * producers;
            const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(full_bar + s), phase, abort_flag, status));
            if (!ok) break;
            __syncwarp();
            if ((threadIdx.x & 31) == 0) mbar_arrive(smem_u32(empty_bar + s));
            if (++j == per) { j = 0; phase ^= 1u; }
        }
    }
}

}  // namespace
}  // namespace q8

extern "C" q8_status q8_measure_l2_operand_peak(const void *buf, int64_t rows, int64_t K, int boxes_per_sm, int sms_used,
                                                int producers, double *gbs, double *elapsed_ms, void *stream)
{
    using namespace q8;
    if (buf == nullptr || gbs == nullptr) return Q8_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(buf) & 15u) != 0) return Q8_ERR_ALIGN;
    if (rows < kBoxRows || rows % kBoxRows != 0 || K < BLOCK_K || K % BLOCK_K != 0 || boxes_per_sm < 1 ||
        boxes_per_sm > (1 << 20) || sms_used < 0 || sms_used > sm_count() || producers < 1 ||
        producers > kMaxProducers || kRing % producers != 0)
        return Q8_ERR_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CUtensorMap map;
    if (!make_tmap(&map, static_cast<const int8_t *>(buf), rows, K, kBoxRows)) return Q8_ERR_CUDA;
    if (cudaFuncSetAttribute(l2_operand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
        return Q8_ERR_CUDA;
    int32_t *status = nullptr;
    if (cudaMalloc(&status, sizeof(int32_t)) != cudaSuccess) return Q8_ERR_CUDA;
    cudaMemsetAsync(status, 0, sizeof(int32_t), s);
    const int sms = sms_used > 0 ? sms_used : sm_count();
    const int64_t boxes_k = K / BLOCK_K, num_boxes = boxes_k * (rows / kBoxRows);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    q8_status result = Q8_OK;
    float ms = 0.0f;
    int32_t host_status = 0;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) result = Q8_ERR_CUDA;
    if (result == Q8_OK) {
        l2_operand_kernel<<<sms, kThreadsL2, kSmem, s>>>(map, boxes_k, num_boxes, boxes_per_sm, producers, status);  // warm-up: fills L2
        cudaEventRecord(e0, s);
        l2_operand_kernel<<<sms, kThreadsL2, kSmem, s>>>(map, boxes_k, num_boxes, boxes_per_sm, producers, status);
        if (cudaGetLastError() != cudaSuccess || cudaEventRecord(e1, s) != cudaSuccess ||
            cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || !(ms > 0.0f) ||
            cudaMemcpy(&host_status, status, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
            result = Q8_ERR_CUDA;
        else if (host_status != 0)
            result = Q8_ERR_TIMEOUT;
    }
    if (result == Q8_OK) {
        *gbs = (double)sms * boxes_per_sm * kBoxBytes / (ms * 1e-3) / 1e9;
        if (elapsed_ms) *elapsed_ms = ms;
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(status);
    return result;
}
