// q8_linear_noalloc: the quantised FC layer for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc (or any allocating routine) at the point where
// they run a layer: code inside a latency-critical serving loop whose memory was carved up at start-up,
// a plugin that is handed raw device pointers by an engine that owns every allocation, or a process
// whose allocator is locked down after initialisation.  q8_linear needs scratch (the Int8 copy of the
// activation plus a status word), which those callers have nowhere to take from.  This entry point keeps
// that scratch in a fixed array that is part of the loaded library image on every GPU, so the call
// itself allocates nothing.

//
// "Allocates nothing" describes the call itself once the library is warm on a device.  The first call on a
// device (and the first call of each GEMM tile configuration) makes the CUDA runtime load the kernels and this
// array onto that device and sets per-kernel attributes, which the runtime may serve with allocations of its
// own; hosts with a frozen allocator should therefore issue one warm-up call per device and shape class during
// initialisation.  The cached device addresses do not survive cudaDeviceReset.

#include <atomic>

#include "q8_internal.cuh"

namespace {

// 256-byte header (status word, dynamic scale) + room for M*K <= 16 Mi quantised activation bytes.
constexpr size_t kStaticScratchBytes = 256 + (size_t)Q8_NOALLOC_MAX_MK;

// Lives in device memory of every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a stand-in for the symbol; the device address has to be asked
// for, once per device, with that device current.
// Host threads may race to fill an entry; they all obtain the same address, so a plain atomic store suffices.
std::atomic<void *> g_scratch_addr[64];

q8_status static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return Q8_ERR_CUDA;
    void *p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return Q8_ERR_CUDA;
        g_scratch_addr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return Q8_OK;
}

}  // namespace

extern "C" q8_status q8_linear_noalloc(const float *X, const int8_t *Wq, const float *S_w, const float *S_x,
                                       const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K,
                                       int8_t *dbg_Xq, int32_t *dbg_acc, void **status_word, void *stream)
{
    if (M > 0 && K > 0 && (M > (int64_t)Q8_NOALLOC_MAX_MK || K > (int64_t)Q8_NOALLOC_MAX_MK ||
                           M * K > (int64_t)Q8_NOALLOC_MAX_MK))
        return Q8_ERR_WORKSPACE;  // the fixed scratch cannot hold this activation
    void *scratch = nullptr;
    q8_status st = static_scratch(&scratch);
    if (st != Q8_OK) return st;
    if (status_word) *status_word = scratch;  // the status word sits at offset 0 of the scratch
    // linear_impl starts the status word (and, with a dynamic scale, the scale words) at zero in every call and
    // overwrites the quantised activation, so nothing of the previous call's contents is read.
    return q8::linear_impl(X, Wq, S_w, S_x, bias, act, Y, M, N, K, scratch, kStaticScratchBytes, dbg_Xq, dbg_acc,
                           stream, false);
}
