// Self-test of the bounded mbarrier wait (ptx::mbar_wait) that every tensor-core kernel of the library relies on
// to stay interruptible: a wait that can never be satisfied must give up after its limit, raise Q8_ERR_TIMEOUT in
// the status word, set the CTA's abort flag and let the kernel return normally.  The kernel below does exactly
// that and nothing else: no tensor-core work, no copies in flight, nothing that waits without a limit.

#include "q8_internal.cuh"
#include "q8_sm100_ptx.cuh"

namespace q8 {
namespace {

__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(uint64_t limit_ns, int32_t *status, int32_t *report)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar), 1);  // one arrival expected; nobody will ever arrive
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0)  // the waiter: phase 0 has not completed, so waiting for parity 0 cannot succeed
        ok = ptx::mbar_wait(ptx::smem_u32(&bar), 0u, &abort_flag, status, limit_ns);
    __syncthreads();
    // the second warp plays a role that notices the abort through the shared flag, as the roles of the GEMM do
    if (threadIdx.x == 32 && report != nullptr) report[1] = *reinterpret_cast<volatile int *>(&abort_flag);
    if (threadIdx.x == 0 && report != nullptr) report[0] = ok ? 0 : 1;
}

}  // namespace
}  // namespace q8

extern "C" q8_status q8_selftest_wait_timeout(uint64_t limit_ns, int32_t *dev_status, int32_t *dev_report, void *stream)
{
    if (dev_status == nullptr) return Q8_ERR_NULL;
    if (limit_ns < 1000ull || limit_ns > 100000000ull) return Q8_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_status) & 3u) || (reinterpret_cast<uintptr_t>(dev_report) & 3u)) return Q8_ERR_ALIGN;
    q8::wait_timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(limit_ns, dev_status, dev_report);
    return cudaGetLastError() == cudaSuccess ? Q8_OK : Q8_ERR_CUDA;
}
