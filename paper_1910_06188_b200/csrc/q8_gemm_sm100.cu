// Int8 x Int8 -> Int32 GEMM with the fused Q8BERT epilogue on Blackwell tensor cores (sm_100a).
//
// Sec. 3 (inference mode): acc = X_q W_q^T in Int32, accumulated onto the Int32 bias, then
// dequantised by 1 / (S_x S_w) and optionally passed through GELU, all inside one kernel:
//
//   warp 0      TMA producer: 128-byte-swizzled K-major tiles of X_q [M,K] and W_q [N,K] go
//               global -> shared through a ring of mbarrier-guarded stages
//   warp 1      MMA issuer: one lane issues tcgen05.mma kind::i8 (128 x BLOCK_N x 32 per
//               instruction); Int32 accumulators live in TMEM, double buffered
//   warps 2..   epilogue: tcgen05.ld the accumulator, add b_q, convert, scale, GELU, store fp32
//
// The kernel is persistent (one CTA per SM walks a static tile list), so the epilogue of tile i
// overlaps the main loop of tile i+1.  No cluster multicast is used anywhere.  Every wait on an
// mbarrier is bounded: after ~2 s the CTA raises Q8_ERR_TIMEOUT in the status word, all roles
// leave their loops, in-flight copies are drained and TMEM is released before the CTA exits.

#include <cuda.h>

#include "q8_internal.cuh"

namespace q8 {

namespace {

constexpr int BLOCK_M = 128;      // UMMA M (cta_group::1): accumulator row i <-> TMEM lane i
constexpr int BLOCK_K = 128;      // bytes == int8 elements per stage row: one 128-byte swizzle span
constexpr int UMMA_K = 32;        // K of one kind::i8 instruction
constexpr int kAccStages = 2;     // TMEM accumulator double buffering
constexpr int kEpilogueWarps = 4; // one per TMEM lane quarter
constexpr int kThreads = 64 + 32 * kEpilogueWarps;
constexpr uint64_t kWaitLimitNs = 2000000000ull;

template <int BLOCK_N>
struct Cfg {
    static constexpr int kABytes = BLOCK_M * BLOCK_K;
    static constexpr int kBBytes = BLOCK_N * BLOCK_K;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = (192 * 1024) / kStageBytes > 8 ? 8 : (192 * 1024) / kStageBytes;
    static constexpr int kTmemCols = kAccStages * BLOCK_N < 32 ? 32 : kAccStages * BLOCK_N;
    static constexpr int kBiasBytes = kEpilogueWarps * BLOCK_N * 4;  // one private b_q copy per epilogue warp
    static constexpr int kBarrierBytes = (2 * kStages + 2 * kAccStages) * 8 + 16;
    // +1024: the dynamic shared window is only 16-byte aligned; tiles need 1024 (swizzle atom)
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kBiasBytes + kBarrierBytes;
    static_assert((kTmemCols & (kTmemCols - 1)) == 0 && kTmemCols <= 512, "TMEM columns: power of two <= 512");
    static_assert(BLOCK_N % 16 == 0 && BLOCK_N >= 16 && BLOCK_N <= 256, "UMMA N for M = 128");
    // Instruction descriptor of tcgen05.mma kind::i8: D = S32, A = B = signed 8-bit, both K-major.
    static constexpr uint32_t kInstrDesc = (2u << 4)                           // D format: S32
                                           | (1u << 7)                         // A format: signed int8
                                           | (1u << 10)                        // B format: signed int8
                                           | ((uint32_t)(BLOCK_N >> 3) << 17)  // N / 8
                                           | ((uint32_t)(BLOCK_M >> 4) << 24); // M / 16
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one timed out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                          uint64_t limit_ns = kWaitLimitNs)
{
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
#pragma unroll 1
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            if (status) atomicOr(status, 1 << Q8_ERR_TIMEOUT);
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t c_inner, int32_t c_outer,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c_inner), "r"(c_outer), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, signed 8-bit operands, Int32 accumulate.
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                        uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// mbarrier arrives once every tcgen05 operation issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows 128 bytes apart, 8-row
// groups 1024 bytes apart (stride byte offset); the leading byte offset is unused for this layout.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (base + i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------ the kernel
template <int BLOCK_N>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, GemmArgs a)
{
    using C = Cfg<BLOCK_N>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *smem_a = smem;
    uint8_t *smem_b = smem + C::kStages * C::kABytes;
    int32_t *smem_bq = reinterpret_cast<int32_t *>(smem + C::kStages * C::kStageBytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(smem_bq) + C::kBiasBytes);
    uint64_t *full_bar = bars;
    uint64_t *empty_bar = bars + C::kStages;
    uint64_t *tmem_full_bar = bars + 2 * C::kStages;
    uint64_t *tmem_empty_bar = tmem_full_bar + kAccStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tmem_empty_bar + kAccStages);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t tiles_n = (a.N + BLOCK_N - 1) / BLOCK_N;
    const int64_t tiles_m = (a.M + BLOCK_M - 1) / BLOCK_M;
    const int64_t num_tiles = tiles_m * tiles_n;
    const int num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), 1);
        }
        for (int s = 0; s < kAccStages; ++s) {
            mbar_init(smem_u32(tmem_full_bar + s), 1);
            mbar_init(smem_u32(tmem_empty_bar + s), kEpilogueWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            int issued = 0;  // k-blocks issued so far (for the drain on abort)
            bool ok = true;
            for (int64_t tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int32_t m0 = (int32_t)((tile / tiles_n) * BLOCK_M);
                const int32_t n0 = (int32_t)((tile % tiles_n) * BLOCK_N);
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(smem_u32(empty_bar + s), phase ^ 1u, abort_flag, a.status);
                    if (!ok) break;
                    const uint32_t fb = smem_u32(full_bar + s);
                    mbar_expect_tx(fb, C::kStageBytes);
                    tma_load_2d(smem_u32(smem_a + s * C::kABytes), &tmap_x, kb * BLOCK_K, m0, fb);
                    tma_load_2d(smem_u32(smem_b + s * C::kBBytes), &tmap_w, kb * BLOCK_K, n0, fb);
                    ++issued;
                    if (++s == C::kStages) { s = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // Aborting: let the copies already issued land before the CTA gives up its shared memory.
                const int pending = issued < C::kStages ? issued : C::kStages;
                for (int i = 0; i < pending; ++i) {
                    const int k = issued - 1 - i;  // the i-th most recent k-block
                    const int st = k % C::kStages;
                    const uint32_t par = (uint32_t)((k / C::kStages) & 1);
                    const uint64_t t0 = global_timer_ns();
                    while (!mbar_try_wait(smem_u32(full_bar + st), par) && global_timer_ns() - t0 < 50000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            int as = 0;
            uint32_t aphase = 0;
            bool ok = true;
            bool committed = false;
            int last_as = 0;
            uint32_t last_aphase = 0;
            for (int64_t tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                ok = mbar_wait(smem_u32(tmem_empty_bar + as), aphase ^ 1u, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(as * BLOCK_N);
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(smem_u32(full_bar + s), phase, abort_flag, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t da = smem_desc_sw128(smem_u32(smem_a + s * C::kABytes));
                    const uint64_t db = smem_desc_sw128(smem_u32(smem_b + s * C::kBBytes));
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                        // +32 bytes along K inside the swizzle span == +2 in the (addr >> 4) field
                        umma_i8(tmem_d, da + (uint64_t)(k * (UMMA_K >> 4)), db + (uint64_t)(k * (UMMA_K >> 4)),
                                C::kInstrDesc, (uint32_t)((kb | k) != 0));
                    }
                    umma_commit(smem_u32(empty_bar + s));  // frees the stage once these MMAs have read it
                    if (++s == C::kStages) { s = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(smem_u32(tmem_full_bar + as));  // accumulator complete
                committed = true;
                last_as = as;
                last_aphase = aphase;
                if (++as == kAccStages) { as = 0; aphase ^= 1u; }
            }
            if (!ok && committed) {
                // Aborting: wait (bounded) for the tensor core to finish what was issued.
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(tmem_full_bar + last_as), last_aphase) &&
                       global_timer_ns() - t0 < 50000000ull) {}
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int ew = warp - 2;            // 0 .. kEpilogueWarps-1
        const int quarter = warp & 3;       // TMEM lanes this warp may touch: 32*quarter .. +31
        const float S_out = __fmul_rn(__ldg(a.S_x), __ldg(a.S_w));
        const float inv = __fdiv_rn(1.0f, S_out);
        const bool vec_ok = ((a.N & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.Y) & 15u) == 0);
        const bool dbg_vec = a.dbg_acc && ((a.N & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.dbg_acc) & 15u) == 0);
        int as = 0;
        uint32_t aphase = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            const int64_t m0 = (tile / tiles_n) * BLOCK_M;
            const int64_t n0 = (tile % tiles_n) * BLOCK_N;
            // b_q for this tile's columns (Sec. 3: bias quantised at S_x * S_w).  Each warp keeps its own
            // copy, so the epilogue warps never have to wait for one another.
            int32_t *bq = smem_bq + ew * BLOCK_N;
            __syncwarp();
            for (int c = lane; c < BLOCK_N; c += 32) {
                const int64_t n = n0 + c;
                bq[c] = (a.bias != nullptr && n < a.N) ? quantize_bias(__ldg(a.bias + n), S_out) : 0;
            }
            __syncwarp();
            ok = mbar_wait(smem_u32(tmem_full_bar + as), aphase, abort_flag, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int64_t row = m0 + quarter * 32 + lane;
            const bool row_ok = row < a.M;
            float *yrow = a.Y + row * a.N;
            int32_t *drow = a.dbg_acc ? a.dbg_acc + row * a.N : nullptr;
#pragma unroll 1
            for (int c0 = 0; c0 < BLOCK_N; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(as * BLOCK_N + c0), r);
                tmem_ld_wait();
                if (n0 + c0 >= a.N) continue;  // warp-uniform
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const int64_t n = n0 + c0 + 4 * g;
                    int32_t v[4];
                    float y[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        v[j] = add_wrap((int32_t)r[4 * g + j], bq[c0 + 4 * g + j]);
                        y[j] = finish_output(v[j], inv, a.act);
                    }
                    if (!row_ok) continue;
                    if (vec_ok) {
                        if (n < a.N) *reinterpret_cast<float4 *>(yrow + n) = make_float4(y[0], y[1], y[2], y[3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (n + j < a.N) yrow[n + j] = y[j];
                    }
                    if (drow) {
                        if (dbg_vec) {
                            if (n < a.N) *reinterpret_cast<int4 *>(drow + n) = make_int4(v[0], v[1], v[2], v[3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                if (n + j < a.N) drow[n + j] = v[j];
                        }
                    }
                }
            }
            // hand the accumulator buffer back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(tmem_empty_bar + as));
            if (++as == kAccStages) { as = 0; aphase ^= 1u; }
        }
    }

    // ---------------- teardown (reached by every thread, also when aborting) ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Row-major int8 matrix [rows, K] as a 2-D tensor map with (128 x box_rows) boxes, 128-byte swizzle.
// Elements outside the matrix read as zero, which is what ragged M, N and K tails need.
bool make_tmap(CUtensorMap *map, const int8_t *base, int64_t rows, int64_t K, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {(cuuint32_t)BLOCK_K, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int sm_count()
{
    static int n = [] {
        int dev = 0, v = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

template <int BLOCK_N>
cudaError_t launch_cfg(const GemmArgs &a, cudaStream_t s)
{
    using C = Cfg<BLOCK_N>;
    static bool attr_set[64] = {};  // the opt-in shared-memory size is a per-device, per-function attribute
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(gemm_tcgen05_kernel<BLOCK_N>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 C::kSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    CUtensorMap tx, tw;
    if (!make_tmap(&tx, a.Xq, a.M, a.K, BLOCK_M) || !make_tmap(&tw, a.Wq, a.N, a.K, BLOCK_N))
        return cudaErrorInvalidValue;
    const int64_t tiles = ((a.M + BLOCK_M - 1) / BLOCK_M) * ((a.N + BLOCK_N - 1) / BLOCK_N);
    const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    gemm_tcgen05_kernel<BLOCK_N><<<grid, kThreads, C::kSmemBytes, s>>>(tx, tw, a);
    LaunchInfo &li = last_launch_info();
    li.gemm_kernel = 1;
    li.block_n = BLOCK_N;
    li.grid = grid;
    li.launches += 1;
    return cudaGetLastError();
}

// Relative time of one 32-deep K step of a 128 x bn tile: the tensor pipe needs bn/2 cycles, reading
// the (128 + bn) x 32 operand bytes from shared memory needs (128 + bn)/4; plus a fixed per-step cost.
double tile_step_cost(int bn)
{
    const double mma = bn / 2.0, smem = (128 + bn) / 4.0;
    return (mma > smem ? mma : smem) + 8.0;
}

}  // namespace

bool tcgen05_gemm_supported(const GemmArgs &a)
{
    return (a.K % 16 == 0) && ((reinterpret_cast<uintptr_t>(a.Xq) & 15u) == 0) &&
           ((reinterpret_cast<uintptr_t>(a.Wq) & 15u) == 0) && a.M < (int64_t(1) << 31) && a.N < (int64_t(1) << 31);
}

cudaError_t launch_gemm_tcgen05(const GemmArgs &a, cudaStream_t s)
{
    const int sms = sm_count();
    const int64_t tm = (a.M + BLOCK_M - 1) / BLOCK_M;
    // Pick the tile width that minimises (waves over the SMs) x (time of one tile).
    int best = 32;
    double best_cost = 0.0;
    for (int bn : {256, 128, 64, 32}) {
        if (bn > 32 && bn / 2 >= a.N) continue;  // more than half of the tile would be padding
        const int64_t tiles = tm * ((a.N + bn - 1) / bn);
        const double cost = (double)((tiles + sms - 1) / sms) * tile_step_cost(bn);
        if (best_cost == 0.0 || cost < best_cost) {
            best = bn;
            best_cost = cost;
        }
    }
    switch (best) {
        case 256: return launch_cfg<256>(a, s);
        case 128: return launch_cfg<128>(a, s);
        case 64: return launch_cfg<64>(a, s);
        default: return launch_cfg<32>(a, s);
    }
}

}  // namespace q8
