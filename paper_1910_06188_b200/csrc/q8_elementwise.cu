// HBM-bound kernels of the Q8BERT inference path: max|x| reduction (Eq. 3 / Eq. 4 / Sec. 4.1),
// the quantiser of Eq. 1, the EMA update of Eq. 4 and the Int8 embedding gather of Sec. 3.
//
// All of them stream their input once with 16-byte loads and stores; the grid is a multiple of
// the SM count with a grid-stride loop so every SM keeps several independent loads in flight.

#include "q8_internal.cuh"

namespace q8 {

namespace {

constexpr int kThreads = 256;

int sm_count()
{
    static int n = [] {
        int dev = 0, v = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

int grid_for(int64_t work_items, int items_per_block, int blocks_per_sm)
{
    int64_t want = (work_items + items_per_block - 1) / items_per_block;
    int64_t cap = (int64_t)sm_count() * blocks_per_sm;
    if (want < 1) want = 1;
    return (int)(want < cap ? want : cap);
}

// ------------------------------------------------------------------ max|x|
__device__ __forceinline__ float absmax4(float m, float4 v)
{
    // fmaxf drops a NaN operand, so NaN entries are skipped; +-Inf propagates.
    m = fmaxf(m, fabsf(v.x));
    m = fmaxf(m, fabsf(v.y));
    m = fmaxf(m, fabsf(v.z));
    return fmaxf(m, fabsf(v.w));
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads) absmax_kernel(const float *__restrict__ x, int64_t n,
                                                          uint32_t *__restrict__ bits)
{
    float m = 0.0f;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    if (VEC) {
        const float4 *x4 = reinterpret_cast<const float4 *>(x);
        const int64_t n4 = n >> 2;
        int64_t i = tid;
        // four independent 16-byte loads per iteration
        for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
            float4 a = __ldg(x4 + i), b = __ldg(x4 + i + nthreads), c = __ldg(x4 + i + 2 * nthreads),
                   d = __ldg(x4 + i + 3 * nthreads);
            m = absmax4(absmax4(absmax4(absmax4(m, a), b), c), d);
        }
        for (; i < n4; i += nthreads) m = absmax4(m, __ldg(x4 + i));
        for (int64_t j = (n4 << 2) + tid; j < n; j += nthreads) m = fmaxf(m, fabsf(x[j]));
    } else {
        for (int64_t j = tid; j < n; j += nthreads) m = fmaxf(m, fabsf(x[j]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    __shared__ float warp_max[kThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0.0f;
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        // non-negative floats (and +Inf) order like their bit patterns
        if (threadIdx.x == 0 && m > 0.0f) atomicMax(bits, __float_as_uint(m));
    }
}

// S = 127 / max|.| (Eq. 3), in place over the scratch word when bits and S alias.
__global__ void scale_from_absmax_kernel(const uint32_t *bits, float *S, int32_t *status)
{
    float a = __uint_as_float(*bits);
    float s;
    if (!(a > 0.0f) || isinf(a)) {
        s = 1.0f;
        if (status) atomicOr(status, 1 << Q8_ERR_SCALE);
    } else {
        s = __fdiv_rn(127.0f, a);
    }
    *S = s;
}

// ------------------------------------------------------------------ Eq. 1
__device__ __forceinline__ int32_t quantize_one(float x, float S) { return quantize_value(x, S); }

__device__ __forceinline__ uint32_t quantize_pack4(float4 v, float S) { return q8::quantize_pack4(v.x, v.y, v.z, v.w, S); }

// VEC: a thread turns one 16-byte load (4 floats) into one 4-byte store, four of them in flight
// per iteration; consecutive lanes touch consecutive addresses on both sides.
// With absmax_bits (dynamic scale, Sec. 4.1) every thread derives S = 127 / max|x| from the finished abs-max word
// itself (one correctly rounded division, the same value in every thread) and thread 0 of the grid publishes it
// in *S_out for the GEMM that follows, so no separate scale kernel runs; otherwise S is read from S_ptr.
template <bool VEC>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const float *__restrict__ x, int64_t n,
                                                            const float *__restrict__ S_ptr,
                                                            int8_t *__restrict__ xq, int8_t *__restrict__ xq_copy,
                                                            const uint32_t *__restrict__ absmax_bits = nullptr,
                                                            float *__restrict__ S_out = nullptr,
                                                            int32_t *__restrict__ status = nullptr,
                                                            int32_t *__restrict__ clear_word = nullptr)
{
    grid_dependency_release_next(n <= kSmallProblemElems);
    grid_dependency_wait();
    // first kernel of a static-scale q8_linear call: start the call's status word at zero
    if (clear_word != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *clear_word = 0;
    float S;
    if (absmax_bits != nullptr) {
        const float a = __uint_as_float(__ldg(absmax_bits));
        const bool bad = !(a > 0.0f) || isinf(a);
        S = bad ? 1.0f : __fdiv_rn(127.0f, a);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            *S_out = S;
            if (bad && status) atomicOr(status, 1 << Q8_ERR_SCALE);
        }
    } else {
        S = __ldg(S_ptr);
        // a caller-supplied scale (an Eq. 4 result) that is zero, negative or not finite cannot quantise anything
        // meaningful: the call still runs, and the condition is reported like a bad derived scale
        if (blockIdx.x == 0 && threadIdx.x == 0 && (!(S > 0.0f) || isinf(S))) {
            int32_t *word = status != nullptr ? status : clear_word;
            if (word != nullptr) atomicOr(word, 1 << Q8_ERR_SCALE);
        }
    }
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    if (VEC) {
        const float4 *x4 = reinterpret_cast<const float4 *>(x);
        uint32_t *q4 = reinterpret_cast<uint32_t *>(xq);
        uint32_t *c4 = reinterpret_cast<uint32_t *>(xq_copy);
        const int64_t n4 = n >> 2;
        int64_t i = tid;
        for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
            float4 a = __ldg(x4 + i), b = __ldg(x4 + i + nthreads), c = __ldg(x4 + i + 2 * nthreads),
                   d = __ldg(x4 + i + 3 * nthreads);
            uint32_t qa = quantize_pack4(a, S), qb = quantize_pack4(b, S), qc = quantize_pack4(c, S),
                     qd = quantize_pack4(d, S);
            q4[i] = qa;
            q4[i + nthreads] = qb;
            q4[i + 2 * nthreads] = qc;
            q4[i + 3 * nthreads] = qd;
            if (xq_copy) {
                c4[i] = qa;
                c4[i + nthreads] = qb;
                c4[i + 2 * nthreads] = qc;
                c4[i + 3 * nthreads] = qd;
            }
        }
        for (; i < n4; i += nthreads) {
            uint32_t q = quantize_pack4(__ldg(x4 + i), S);
            q4[i] = q;
            if (xq_copy) c4[i] = q;
        }
        for (int64_t j = (n4 << 2) + tid; j < n; j += nthreads) {
            int8_t q = (int8_t)quantize_one(x[j], S);
            xq[j] = q;
            if (xq_copy) xq_copy[j] = q;
        }
    } else {
        for (int64_t j = tid; j < n; j += nthreads) {
            int8_t q = (int8_t)quantize_one(x[j], S);
            xq[j] = q;
            if (xq_copy) xq_copy[j] = q;
        }
    }
}

// Dynamic scale and Eq. 1 in ONE launch for a small activation (Sec. 4.1; e.g. one 128-token batch): a single
// cluster of 8 CTAs holds the whole tensor in registers (up to 12 float4 per thread), so the tensor is read once.
// Each CTA reduces max|x| of its share, the 8 partial maxima are exchanged through distributed shared memory
// (one cluster barrier), every thread derives the same S = 127 / max|x| and quantises the values it holds.
// CTA 0 publishes S and sets the call's status word (0, or the Q8_ERR_SCALE bit for a zero / infinite maximum).
constexpr int kDqCluster = 8, kDqThreads = 512, kDqVecPerThread = 12;
constexpr int64_t kDqMaxElems = (int64_t)kDqCluster * kDqThreads * kDqVecPerThread * 4;  // 196608 = 256 x 768

__global__ void __launch_bounds__(kDqThreads) quantize_dynamic_cluster_kernel(const float *__restrict__ x, int64_t n,
                                                                              float *__restrict__ S_out,
                                                                              int32_t *__restrict__ status,
                                                                              int8_t *__restrict__ xq,
                                                                              int8_t *__restrict__ xq_copy)
{
    grid_dependency_release_next(true);  // small by construction
    grid_dependency_wait();
    __shared__ float warp_max[kDqThreads / 32];
    __shared__ float cta_max, all_max;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int64_t n4 = n >> 2;  // n % 4 == 0 (checked by the host)
    const float4 *x4 = reinterpret_cast<const float4 *>(x);
    const int64_t first = (int64_t)rank * kDqThreads + threadIdx.x;
    constexpr int64_t kStride = (int64_t)kDqCluster * kDqThreads;
    float4 v[kDqVecPerThread];
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < kDqVecPerThread; ++i) {
        const int64_t idx = first + i * kStride;
        v[i] = idx < n4 ? __ldg(x4 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        m = absmax4(m, v[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < kDqThreads / 32 ? warp_max[threadIdx.x] : 0.0f;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (threadIdx.x == 0) cta_max = m;
    }
    // every CTA's partial maximum is in place before any CTA reads its peers'
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (threadIdx.x < 32) {
        float p = 0.0f;
        if (threadIdx.x < kDqCluster) {
            uint32_t remote;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                         : "=r"(remote)
                         : "r"((uint32_t)__cvta_generic_to_shared(&cta_max)), "r"((uint32_t)threadIdx.x));
            asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(p) : "r"(remote) : "memory");
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) p = fmaxf(p, __shfl_xor_sync(0xffffffffu, p, o));
        if (threadIdx.x == 0) all_max = p;
    }
    // no CTA may exit (and give up its shared memory) while a peer can still read it
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    __syncthreads();
    const float a = all_max;
    const bool bad = !(a > 0.0f) || isinf(a);
    const float S = bad ? 1.0f : __fdiv_rn(127.0f, a);
    if (rank == 0 && threadIdx.x == 0) {
        *S_out = S;
        if (status) *status = bad ? (1 << Q8_ERR_SCALE) : 0;  // first kernel of the call: starts the status word
    }
    uint32_t *q4 = reinterpret_cast<uint32_t *>(xq);
    uint32_t *c4 = reinterpret_cast<uint32_t *>(xq_copy);
#pragma unroll
    for (int i = 0; i < kDqVecPerThread; ++i) {
        const int64_t idx = first + i * kStride;
        if (idx < n4) {
            const uint32_t q = quantize_pack4(v[i], S);
            q4[idx] = q;
            if (xq_copy) c4[idx] = q;
        }
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ------------------------------------------------------------------ Eq. 4
__global__ void ema_update_kernel(CalibState *st, float decay)
{
    float m = __uint_as_float(st->scratch_bits);
    st->scratch_bits = 0u;
    float ema;
    if (st->n_batches == 0 || decay == 0.0f) {
        ema = m;  // first batch, or no history kept: exactly this batch's maximum (the dynamic scale of Sec. 4.1)
    } else {
        // ema += (1 - d) * (m - ema), each operation rounded separately (no fused multiply-add)
        float one_minus_d = __fsub_rn(1.0f, decay);
        float step = __fmul_rn(one_minus_d, __fsub_rn(m, st->ema));
        ema = __fadd_rn(st->ema, step);
    }
    st->ema = ema;
    st->n_batches += 1;
    if (!(ema > 0.0f) || isinf(ema)) {
        st->S_x = 1.0f;
        st->status |= 1 << Q8_ERR_SCALE;
    } else {
        st->S_x = __fdiv_rn(127.0f, ema);
    }
}

// ------------------------------------------------------------------ Int8 embedding (Sec. 3)
__device__ __forceinline__ float4 dequant4(uint32_t w, float inv)
{
    float4 f;
    f.x = __fmul_rn((float)(int8_t)(w & 0xffu), inv);
    f.y = __fmul_rn((float)(int8_t)((w >> 8) & 0xffu), inv);
    f.z = __fmul_rn((float)(int8_t)((w >> 16) & 0xffu), inv);
    f.w = __fmul_rn((float)(int8_t)(w >> 24), inv);
    return f;
}

// VEC: a CTA walks token rows (four at a time, so four independent gathers are in flight per thread);
// within a row one thread moves 4 table bytes (one 4-byte load) to one 16-byte streaming store, so a
// warp reads 128 and writes 512 contiguous bytes.  No per-element index arithmetic beyond adds.
template <bool VEC>
__global__ void __launch_bounds__(kThreads) embedding_kernel(const int32_t *__restrict__ ids, int64_t T,
                                                             const int8_t *__restrict__ Eq,
                                                             const float *__restrict__ S_e, int64_t V, int64_t H,
                                                             float *__restrict__ out, int8_t *__restrict__ rows_q,
                                                             int32_t *__restrict__ status)
{
    grid_dependency_release_next(T * H <= kSmallProblemElems);
    grid_dependency_wait();
    const float inv = __fdiv_rn(1.0f, __ldg(S_e));
    if (VEC) {
        const int per_row = (int)(H >> 2);
        for (int64_t t0 = (int64_t)blockIdx.x * 4; t0 < T; t0 += (int64_t)gridDim.x * 4) {
            int64_t id[4];
            bool ok[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                id[r] = (t0 + r < T) ? (int64_t)__ldg(ids + t0 + r) : -1;
                ok[r] = id[r] >= 0 && id[r] < V;
                if (!ok[r] && t0 + r < T && threadIdx.x == 0 && status) atomicOr(status, 1 << Q8_ERR_INDEX);
            }
            for (int c = threadIdx.x; c < per_row; c += blockDim.x) {
                uint32_t q[4];
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    q[r] = ok[r] ? __ldg(reinterpret_cast<const uint32_t *>(Eq + id[r] * H) + c) : 0u;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (t0 + r >= T) break;
                    __stcs(reinterpret_cast<float4 *>(out + (t0 + r) * H) + c, dequant4(q[r], inv));
                    if (rows_q) reinterpret_cast<uint32_t *>(rows_q + (t0 + r) * H)[c] = q[r];
                }
            }
        }
    } else {
        const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
        const int64_t total = T * H;
        for (int64_t e = tid; e < total; e += nthreads) {
            const int64_t t = e / H, h = e - t * H;
            const int64_t id = __ldg(ids + t);
            int8_t q = 0;
            if (id >= 0 && id < V) {
                q = Eq[id * H + h];
            } else if (h == 0 && status) {
                atomicOr(status, 1 << Q8_ERR_INDEX);
            }
            out[e] = __fmul_rn((float)q, inv);
            if (rows_q) rows_q[e] = q;
        }
    }
}

// ------------------------------------------------------------------ training mode: fake quantisation (Sec. 2.2)
// x_hat = Quantize(x | S) / S: the rounding of Eq. 1 simulated in floating point (one fp32 division per element).
__device__ __forceinline__ float fake_one(float x, float S) { return __fdiv_rn((float)quantize_value(x, S), S); }

template <bool VEC>
__global__ void __launch_bounds__(kThreads) fake_quantize_kernel(const float *__restrict__ x, int64_t n,
                                                                 const float *__restrict__ S_ptr,
                                                                 float *__restrict__ xhat)
{
    const float S = __ldg(S_ptr);
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    if (VEC) {
        const float4 *x4 = reinterpret_cast<const float4 *>(x);
        float4 *o4 = reinterpret_cast<float4 *>(xhat);
        const int64_t n4 = n >> 2;
        for (int64_t i = tid; i < n4; i += nthreads) {
            const float4 v = __ldg(x4 + i);
            o4[i] = make_float4(fake_one(v.x, S), fake_one(v.y, S), fake_one(v.z, S), fake_one(v.w, S));
        }
        for (int64_t j = (n4 << 2) + tid; j < n; j += nthreads) xhat[j] = fake_one(x[j], S);
    } else {
        for (int64_t j = tid; j < n; j += nthreads) xhat[j] = fake_one(x[j], S);
    }
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

cudaError_t launch_absmax(const float *x, int64_t n, uint32_t *bits, cudaStream_t s)
{
    if (n <= 0) return cudaSuccess;
    if (aligned16(x)) {
        absmax_kernel<true><<<grid_for(n >> 2, kThreads * 4, 8), kThreads, 0, s>>>(x, n, bits);
    } else {
        absmax_kernel<false><<<grid_for(n, kThreads * 4, 8), kThreads, 0, s>>>(x, n, bits);
    }
    return cudaGetLastError();
}

cudaError_t launch_scale_from_absmax(const uint32_t *bits, float *S, int32_t *status, cudaStream_t s)
{
    scale_from_absmax_kernel<<<1, 1, 0, s>>>(bits, S, status);
    return cudaGetLastError();
}

// Grid of the vectorised quantise pass: CTAs per SM, grid-stride.  Measured on 24576 x 1024 / 24576 x 4096 fp32 inputs
// (graph replays of three passes over separate buffers): 2 CTAs per SM 26.6 / 92.2 us, 3: 23.0 / 78.6, 4: 21.4 / 75.4,
// 5: 25.4 / 89.6, 8: 21.6 / 77.3, 16: 24.8 / 78.4: a power-of-two stride between a thread's successive loads suits
// the memory system best, and four CTAs already keep enough loads in flight (64 KB per SM).
constexpr int kQuantCtasPerSm = 4;

cudaError_t launch_quantize(const float *x, int64_t n, const float *S, int8_t *xq, int8_t *xq_copy, cudaStream_t s,
                            int32_t *clear_word, int32_t *status)
{
    if (n <= 0) return cudaSuccess;
    if (aligned16(x) && aligned16(xq) && (xq_copy == nullptr || aligned16(xq_copy))) {
        return launch_overlapping_tail(quantize_kernel<true>, dim3(grid_for((n + 3) >> 2, kThreads * 4, kQuantCtasPerSm)),
                                       dim3(kThreads), 0, s, x, n, S, xq, xq_copy, nullptr, nullptr, status, clear_word);
    } else {
        quantize_kernel<false><<<grid_for(n, kThreads * 4, 8), kThreads, 0, s>>>(x, n, S, xq, xq_copy, nullptr, nullptr,
                                                                                 status, clear_word);
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_dynamic(const float *x, int64_t n, const uint32_t *absmax_bits, float *S_out, int32_t *status,
                                    int8_t *xq, int8_t *xq_copy, cudaStream_t s, bool clear_status)
{
    if (n <= 0) return cudaSuccess;
    int32_t *clear_word = clear_status ? status : nullptr;
    if (aligned16(x) && aligned16(xq) && (xq_copy == nullptr || aligned16(xq_copy))) {
        return launch_overlapping_tail(quantize_kernel<true>, dim3(grid_for((n + 3) >> 2, kThreads * 4, kQuantCtasPerSm)),
                                       dim3(kThreads), 0, s, x, n, nullptr, xq, xq_copy, absmax_bits, S_out, status, clear_word);
    } else {
        quantize_kernel<false><<<grid_for(n, kThreads * 4, 8), kThreads, 0, s>>>(x, n, nullptr, xq, xq_copy, absmax_bits,
                                                                                 S_out, status, clear_word);
    }
    return cudaGetLastError();
}

bool quantize_dynamic_small_supported(const float *x, int64_t n, const int8_t *xq, const int8_t *xq_copy)
{
    return n > 0 && n <= kDqMaxElems && (n & 3) == 0 && aligned16(x) && aligned16(xq) &&
           (xq_copy == nullptr || aligned16(xq_copy));
}

cudaError_t launch_quantize_dynamic_small(const float *x, int64_t n, float *S_out, int32_t *status, int8_t *xq,
                                          int8_t *xq_copy, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kDqCluster);
    cfg.blockDim = dim3(kDqThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kDqCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, quantize_dynamic_cluster_kernel, x, n, S_out, status, xq, xq_copy);
}

cudaError_t launch_fake_quantize(const float *x, int64_t n, const float *S, float *xhat, cudaStream_t s)
{
    if (n <= 0) return cudaSuccess;
    if (aligned16(x) && aligned16(xhat)) {
        fake_quantize_kernel<true><<<grid_for((n + 3) >> 2, kThreads * 4, 8), kThreads, 0, s>>>(x, n, S, xhat);
    } else {
        fake_quantize_kernel<false><<<grid_for(n, kThreads * 4, 8), kThreads, 0, s>>>(x, n, S, xhat);
    }
    return cudaGetLastError();
}

cudaError_t launch_ema_update(CalibState *st, float decay, cudaStream_t s)
{
    ema_update_kernel<<<1, 1, 0, s>>>(st, decay);
    return cudaGetLastError();
}

cudaError_t launch_embedding(const int32_t *ids, int64_t T, const int8_t *Eq, const float *S_e, int64_t V,
                             int64_t H, float *out, int8_t *rows_q, int32_t *status, cudaStream_t s)
{
    if (T <= 0 || H <= 0) return cudaSuccess;
    const bool vec = (H % 4 == 0) && aligned16(Eq) && aligned16(out) && (rows_q == nullptr || aligned16(rows_q));
    if (vec) {
        // one thread per 4-byte piece of a row, rounded up to whole warps; a CTA takes 4 rows per iteration
        int threads = (int)(((H >> 2) + 31) / 32 * 32);
        if (threads > kThreads) threads = kThreads;
        return launch_overlapping_tail(embedding_kernel<true>, dim3(grid_for((T + 3) / 4, 1, 16)), dim3(threads), 0, s, ids, T,
                                       Eq, S_e, V, H, out, rows_q, status);
    } else {
        embedding_kernel<false><<<grid_for(T * H, kThreads, 8), kThreads, 0, s>>>(ids, T, Eq, S_e, V, H, out,
                                                                                 rows_q, status);
    }
    return cudaGetLastError();
}

}  // namespace q8
