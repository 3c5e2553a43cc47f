// Issue-bound Int8 tensor-core rate of this GPU: the ceiling the GEMM's tensor pipe could reach if operands
// never had to be fetched.
//
// Every SM (CTAS = 1) or SM pair (CTAS = 2, cta_group::2) keeps one operand tile pair resident in shared
// memory, filled once with pseudo-random signed bytes (all-zero operands would draw less power and flatter the
// clock), and one thread issues the same tcgen05.mma kind::i8 shapes as the GEMM kernel (M = 128 * CTAS,
// N = 256, K = 32, four K steps across one 128-byte swizzle span) back to back into two alternating TMEM
// accumulators.  Nothing is loaded by TMA and nothing is stored, so the time is the tensor pipe's own.
// Work is issued in batches; each batch ends in a tcgen05.commit and the issuer waits (bounded) for batch i-1
// only after batch i is queued, so the pipe never drains.

#include "q8_internal.cuh"
#include "q8_sm100_ptx.cuh"

namespace q8 {

namespace {

using namespace ptx;

constexpr int kPeakN = 256;
constexpr int kPeakTmemCols = 512;
constexpr int kTileBytesA = 128 * 128;  // 128 rows x 128 bytes (K-major, one swizzle span wide)

template <int CTAS>
__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int batches, int mmas_per_batch, int32_t *status)
{
    constexpr int kBRows = kPeakN / CTAS;
    constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kPeakN >> 3) << 17) |
                                ((uint32_t)((128 * CTAS) >> 4) << 24);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *smem_a = tiles, *smem_b = tiles + kTileBytesA;
    __shared__ __align__(8) uint64_t done_bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = CTAS == 2 ? cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;

    // operand bytes: a cheap integer hash of the position, different per CTA
    for (int i = threadIdx.x; i < (kTileBytesA + kBRows * 128) / 4; i += blockDim.x) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u + 12345u;
        h ^= h >> 15;
        h *= 2246822519u;
        h ^= h >> 13;
        reinterpret_cast<uint32_t *>(tiles)[i] = h;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(done_bar + 0), 1);
        mbar_init(smem_u32(done_bar + 1), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_proxy_async_smem();  // the tensor core reads the tiles through the async proxy
    if (warp == 1) {
        if (CTAS == 2) tmem_alloc_pair(smem_u32(&tmem_slot), kPeakTmemCols);
        else tmem_alloc(smem_u32(&tmem_slot), kPeakTmemCols);
    }
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0 && lane == 0 && leader) {
        const uint64_t da = smem_desc_sw128(smem_u32(smem_a)), db = smem_desc_sw128(smem_u32(smem_b));
        bool ok = true;
        for (int b = 0; ok && b < batches; ++b) {
            for (int i = 0; i < mmas_per_batch; ++i) {
                const uint32_t tmem_d = tmem_base + (uint32_t)((i >> 2) & 1) * kPeakN;  // alternate accumulators
                const uint64_t adv = (uint64_t)((i & 3) * 2);                           // +32 bytes along K
                const uint32_t accumulate = i >= 8 ? 1u : 0u;  // each batch starts both accumulators afresh
                if (CTAS == 2) umma_i8_pair(tmem_d, da + adv, db + adv, kIdesc, accumulate);
                else umma_i8(tmem_d, da + adv, db + adv, kIdesc, accumulate);
            }
            if (CTAS == 2) umma_commit_pair(smem_u32(done_bar + (b & 1)));
            else umma_commit(smem_u32(done_bar + (b & 1)));
            // wait for the batch before this one: its barrier is reused two batches later
            if (b >= 1) ok = mbar_wait(smem_u32(done_bar + ((b - 1) & 1)), (uint32_t)(((b - 1) >> 1) & 1), &abort_flag, status);
        }
        if (ok && batches > 0)
            ok = mbar_wait(smem_u32(done_bar + ((batches - 1) & 1)), (uint32_t)(((batches - 1) >> 1) & 1), &abort_flag, status);
        if (!ok && batches > 0) {
            // aborting: give the tensor core a bounded while to finish what is queued before TMEM is freed
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(done_bar + ((batches - 1) & 1)), (uint32_t)(((batches - 1) >> 1) & 1)) &&
                   global_timer_ns() - t0 < 50000000ull) {}
        }
    }

    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if (CTAS == 2) tmem_dealloc_pair(tmem_base, kPeakTmemCols);
        else tmem_dealloc(tmem_base, kPeakTmemCols);
    }
}

template <int CTAS>
cudaError_t launch_peak(int units, int batches, int mmas_per_batch, int32_t *status, cudaStream_t s)
{
    auto kernel = mma_peak_kernel<CTAS>;
    const int smem = 1024 + kTileBytesA + (kPeakN / CTAS) * 128;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * CTAS));
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = CTAS;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, batches, mmas_per_batch, status);
}

}  // namespace

}  // namespace q8

extern "C" q8_status q8_measure_int8_mma_peak(int ctas, double seconds, double *tops, double *elapsed_ms, int *sms_used,
                                              void *dev_status, void *stream)
{
    using namespace q8;
    if ((ctas != 1 && ctas != 2) || !(seconds > 0.0) || seconds > 5.0 || tops == nullptr) return Q8_ERR_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return Q8_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < ctas) return Q8_ERR_CUDA;
    const int units = sms / ctas;
    int32_t *status = static_cast<int32_t *>(dev_status);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess) return Q8_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) {
        cudaEventDestroy(e0);
        return Q8_ERR_CUDA;
    }
    const int kMmasPerBatch = 256;
    const double ops_per_mma = 2.0 * (128.0 * ctas) * 256.0 * 32.0;
    auto timed = [&](int batches, float *ms) -> cudaError_t {
        cudaError_t e = cudaEventRecord(e0, s);
        if (e != cudaSuccess) return e;
        e = ctas == 2 ? launch_peak<2>(units, batches, kMmasPerBatch, status, s)
                      : launch_peak<1>(units, batches, kMmasPerBatch, status, s);
        if (e != cudaSuccess) return e;
        e = cudaEventRecord(e1, s);
        if (e != cudaSuccess) return e;
        e = cudaEventSynchronize(e1);
        if (e != cudaSuccess) return e;
        return cudaEventElapsedTime(ms, e0, e1);
    };
    // a short calibration launch sizes the timed one; each launch stays well under the device-side wait limit
    float ms = 0.0f;
    cudaError_t e = timed(64, &ms);
    q8_status result = Q8_OK;
    if (e != cudaSuccess || !(ms > 0.0f)) {
        result = Q8_ERR_CUDA;
    } else {
        double per_batch_ms = ms / 64.0;
        double want = seconds * 1e3 / per_batch_ms;
        int batches = want > 4.0e6 ? 4000000 : (want < 64.0 ? 64 : (int)want);
        e = timed(batches, &ms);
        if (e != cudaSuccess || !(ms > 0.0f)) {
            result = Q8_ERR_CUDA;
        } else {
            *tops = ops_per_mma * (double)kMmasPerBatch * (double)batches * (double)units / (ms * 1e-3) / 1e12;
            if (elapsed_ms) *elapsed_ms = ms;
            if (sms_used) *sms_used = units * ctas;
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return result;
}
