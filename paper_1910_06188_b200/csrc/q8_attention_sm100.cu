// Multi-head self-attention (head dimension 64, no mask) on the Blackwell tensor cores with fp32-grade
// accuracy: both products, Q K^T and P V, run as tcgen05.mma kind::tf32 with every fp32 operand split into
// a TF32-exact high part (x rounded to nearest TF32) and the low remainder (x = hi + lo exactly), and
// the three significant partial products hi*hi + hi*lo + lo*hi are accumulated in fp32 in TMEM.  The dropped
// lo*lo term is below 2^-22 relative per product, i.e. at the rounding level of a plain fp32 dot product.  (The paper keeps attention in fp32 and quantises only the FC layers; this kernel
// is the fp32 attention an encoder forward needs around them.)
//
// One CTA = 128 queries of one (sequence, head); 8 warps.  All operands are staged by the threads themselves
// (global -> registers -> split -> shared memory in the K-major 128-byte-swizzled layout the MMA reads);
// no TMA, no multicast.
//   phase 1  Q tile (scaled by log2(e)/8) -> Q_hi, Q_lo; then per chunk of 64 keys: K chunk -> K_hi, K_lo,
//            24 MMAs (2 swizzle spans x 4 K steps x 3 partial products) -> scores in TMEM columns [64 c, 64 c + 64)
//   phase 2  row maxima straight from TMEM (each row is shared by two threads, one per half of every chunk)
//   phase 3  per chunk: p = 2^(s - max) -> P_hi, P_lo (A operand, keys along K); V chunk transposed -> V_hi,
//            V_lo (B operand); 24 MMAs accumulate O[128 x 64] in the TMEM columns behind the scores
//   phase 4  O / row sum -> ctx (and optionally Int8 at the next layer's scale)
// The whole score row block lives in TMEM (S_pad + 64 <= 512 columns), so the softmax needs no running
// rescale.  Every wait on the MMA barrier is bounded; on a time-out the CTA raises Q8_ERR_TIMEOUT in the
// status word, skips the rest and still frees its TMEM.

#include "q8_internal.cuh"
#include "q8_sm100_ptx.cuh"

namespace q8 {

namespace {

using namespace ptx;

constexpr int kHeadDim = 64;
constexpr int kQTile = 128;   // queries per CTA = TMEM lanes
constexpr int kChunk = 64;    // keys per chunk = N of the score MMA = K extent of one P / V chunk
constexpr int kThreads = 256;
constexpr int kSpanBytesA = kQTile * 128;  // one swizzle span (32 fp32 of K) of a 128-row operand: 16 KB
constexpr int kSpanBytesB = kChunk * 128;  // ... of a 64-row operand: 8 KB
constexpr int kBufQP = 4 * kSpanBytesA;    // {hi, lo} x 2 spans: Q in phase 1, P in phase 3
constexpr int kBufKV = 4 * kSpanBytesB;    // {hi, lo} x 2 spans: K in phase 1, V^T in phase 3
constexpr int kAttnTcSmemBytes = 1024 + kBufQP + kBufKV;

// tcgen05.mma kind::tf32 instruction descriptor: D = F32, A = B = TF32, both K-major, M = 128, N = 64.
constexpr uint32_t kIdescTf32 = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kChunk >> 3) << 17) |
                                ((uint32_t)(kQTile >> 4) << 24);

// Byte offset of the 16-byte piece `piece` (0..7) of row `row` inside one swizzle span (rows of 128 bytes,
// groups of 8 rows 1024 bytes apart, piece index XORed with the row's position in its group).
__device__ __forceinline__ uint32_t sw128_offset(int row, int piece)
{
    return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((piece ^ (row & 7)) << 4));
}

// x = hi + lo with hi = x rounded to nearest TF32 (10 explicit mantissa bits), so |lo| <= 2^-12 |x|; lo has up
// to 12 significant bits, of which the tensor core's truncation of its operands keeps 11: an error below
// 2^-23 |x|.  (Clearing the low bits of x instead would double |lo| and with it that error.)
__device__ __forceinline__ float round_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}
__device__ __forceinline__ void split_tf32(float x, float &hi, float &lo)
{
    hi = round_tf32(x);
    lo = x - hi;  // exact in fp32
}

__device__ __forceinline__ void store_split4(uint8_t *hi_base, uint8_t *lo_base, uint32_t off, float4 v)
{
    float4 h, l;
    split_tf32(v.x, h.x, l.x);
    split_tf32(v.y, h.y, l.y);
    split_tf32(v.z, h.z, l.z);
    split_tf32(v.w, h.w, l.w);
    *reinterpret_cast<float4 *>(hi_base + off) = h;
    *reinterpret_cast<float4 *>(lo_base + off) = l;
}

// The three partial products of one K-major operand pair over two swizzle spans of 32 fp32 each.  The large
// product hi*hi goes to tmem_main and the two small ones to tmem_corr (which may be the same columns): the
// tensor core rounds every accumulation relative to the accumulator's magnitude, so keeping the corrections
// apart leaves one rounding per K step on the long chain instead of three.
__device__ __forceinline__ void issue_split_mma(uint32_t tmem_main, uint32_t tmem_corr, uint32_t a_hi, uint32_t a_lo,
                                                uint32_t a_span_bytes, uint32_t b_hi, uint32_t b_lo, uint32_t b_span_bytes,
                                                bool accumulate)
{
    const bool shared_acc = tmem_main == tmem_corr;
    uint32_t acc_main = accumulate ? 1u : 0u, acc_corr = accumulate ? 1u : 0u;
#pragma unroll
    for (int span = 0; span < 2; ++span) {
        const uint64_t dah = smem_desc_sw128(a_hi + span * a_span_bytes), dal = smem_desc_sw128(a_lo + span * a_span_bytes);
        const uint64_t dbh = smem_desc_sw128(b_hi + span * b_span_bytes), dbl = smem_desc_sw128(b_lo + span * b_span_bytes);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {  // 8 fp32 = 32 bytes of K per instruction: +2 in the (address >> 4) field
            const uint64_t adv = (uint64_t)(2 * ks);
            umma_tf32(tmem_corr, dal + adv, dbh + adv, kIdescTf32, acc_corr);
            umma_tf32(tmem_corr, dah + adv, dbl + adv, kIdescTf32, 1u);
            acc_corr = 1u;
            if (shared_acc) acc_main = 1u;
            umma_tf32(tmem_main, dah + adv, dbh + adv, kIdescTf32, acc_main);
            acc_main = 1u;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const float *__restrict__ qkv, int S, int64_t H, float scale, float *__restrict__ ctx,
                    const float *__restrict__ S_q, int8_t *__restrict__ ctx_q, uint32_t tmem_cols, int32_t *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *qp_hi = smem, *qp_lo = smem + 2 * kSpanBytesA;
    uint8_t *kv_hi = smem + kBufQP, *kv_lo = kv_hi + 2 * kSpanBytesB;
    __shared__ __align__(8) uint64_t mma_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float row_part[2][kQTile];  // per-row partial maxima, then partial sums, of the two column halves

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int quarter = warp & 3, half = warp >> 2;  // TMEM lane quarter this warp may read; its half of every chunk
    const int row = quarter * 32 + lane;             // query row (TMEM lane) of this thread in phases 2-4
    const int q0 = blockIdx.x * kQTile;
    const int64_t head = blockIdx.y, seq = blockIdx.z;
    const int64_t row_pitch = 3 * H;
    const float *base = qkv + seq * (int64_t)S * row_pitch + head * kHeadDim;
    const int chunks = (S + kChunk - 1) / kChunk;
    const int s_pad = chunks * kChunk;

    if (tid == 0) {
        mbar_init(smem_u32(&mma_bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tmem_o = tmem_base + (uint32_t)s_pad;  // O accumulator: 64 columns behind the scores
    // second accumulator for the small partial products of P V, when the allocation has room for it
    const bool two_acc = (uint32_t)(s_pad + 2 * kHeadDim) <= tmem_cols;
    const uint32_t tmem_o_corr = two_acc ? tmem_o + kHeadDim : tmem_o;
    uint32_t bar_phase = 0;
    bool ok = true;

    // Every thread waits for the MMAs committed last; the outcome is made uniform across the CTA.
    auto wait_mma = [&]() {
        bool mine = mbar_wait(smem_u32(&mma_bar), bar_phase, &abort_flag, status);
        bar_phase ^= 1u;
        ok = __syncthreads_and(mine ? 1 : 0) != 0;
        tc_fence_after();
    };

    // ---------------- phase 1: scores = (Q * log2(e)/8) K^T
    // a 16-byte piece c of a [rows x 64] fp32 tile: row c / 16, span (c % 16) / 8, piece (c % 16) % 8
#pragma unroll
    for (int i = 0; i < (kQTile * 16) / kThreads; ++i) {
        const int c = tid + i * kThreads, r = c >> 4, pc = c & 15;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q0 + r < S) v = __ldg(reinterpret_cast<const float4 *>(base + (int64_t)(q0 + r) * row_pitch) + pc);
        v.x *= scale;
        v.y *= scale;
        v.z *= scale;
        v.w *= scale;
        const uint32_t off = (uint32_t)((pc >> 3) * kSpanBytesA) + sw128_offset(r, pc & 7);
        store_split4(qp_hi, qp_lo, off, v);
    }
    float4 kreg[4];
    auto fetch_rows = [&](int j0, int64_t col0) {  // 64 rows (keys) x 64 fp32 starting at column col0 of qkv
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = tid + i * kThreads, r = c >> 4, pc = c & 15;
            kreg[i] = (j0 + r < S) ? __ldg(reinterpret_cast<const float4 *>(base + (int64_t)(j0 + r) * row_pitch + col0) + pc)
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    fetch_rows(0, H);
    for (int kc = 0; kc < chunks && ok; ++kc) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = tid + i * kThreads, r = c >> 4, pc = c & 15;
            store_split4(kv_hi, kv_lo, (uint32_t)((pc >> 3) * kSpanBytesB) + sw128_offset(r, pc & 7), kreg[i]);
        }
        if (kc + 1 < chunks) fetch_rows((kc + 1) * kChunk, H);  // next K chunk, in flight during the MMAs
        fence_proxy_async_smem();  // the writes above become visible to the tensor core (async proxy)
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            issue_split_mma(tmem_base + (uint32_t)(kc * kChunk), tmem_base + (uint32_t)(kc * kChunk), smem_u32(qp_hi), smem_u32(qp_lo), kSpanBytesA,
                            smem_u32(kv_hi), smem_u32(kv_lo), kSpanBytesB, false);
            umma_commit(smem_u32(&mma_bar));
        }
        wait_mma();  // K buffers are free again; after the last chunk all scores are in TMEM
    }

    // ---------------- phase 2: row maxima (a thread reads its row's columns [64 c + 32 half, +32) of every chunk)
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float m = -INFINITY;
    if (ok) {
        for (int kc = 0; kc < chunks; ++kc) {
            uint32_t v[32];
            const int col0 = kc * kChunk + half * 32;
            tmem_ld_32x32(t_row + (uint32_t)col0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (col0 + j < S) m = fmaxf(m, __uint_as_float(v[j]));
        }
    }
    row_part[half][row] = m;
    __syncthreads();
    m = fmaxf(row_part[0][row], row_part[1][row]);
    __syncthreads();  // row_part is reused for the sums

    // ---------------- phase 3: P = 2^(scores - max), O = P V
    float l = 0.0f;
    // V chunk as a 64 x 64 tile of 4 x 4 blocks: thread = (key block kb, feature block fb); the block is
    // transposed in registers so that each feature row of V^T gets 4 consecutive keys (one 16-byte piece)
    const int vkb = tid >> 4, vfb = tid & 15;
    float4 vreg[4];
    auto fetch_v = [&](int j0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = j0 + 4 * vkb + i;
            vreg[i] = (j < S) ? __ldg(reinterpret_cast<const float4 *>(base + (int64_t)j * row_pitch + 2 * H) + vfb)
                              : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    if (ok) fetch_v(0);
    for (int kc = 0; kc < chunks && ok; ++kc) {
        // V^T[d][key]: rows = features (64), K = keys of this chunk (2 spans of 32)
        {
            const int span = vkb >> 3, piece = vkb & 7;  // keys 4 vkb .. 4 vkb + 3 of the chunk
            const float4 t0 = make_float4(vreg[0].x, vreg[1].x, vreg[2].x, vreg[3].x);
            const float4 t1 = make_float4(vreg[0].y, vreg[1].y, vreg[2].y, vreg[3].y);
            const float4 t2 = make_float4(vreg[0].z, vreg[1].z, vreg[2].z, vreg[3].z);
            const float4 t3 = make_float4(vreg[0].w, vreg[1].w, vreg[2].w, vreg[3].w);
            const uint32_t sb = (uint32_t)(span * kSpanBytesB);
            store_split4(kv_hi, kv_lo, sb + sw128_offset(4 * vfb + 0, piece), t0);
            store_split4(kv_hi, kv_lo, sb + sw128_offset(4 * vfb + 1, piece), t1);
            store_split4(kv_hi, kv_lo, sb + sw128_offset(4 * vfb + 2, piece), t2);
            store_split4(kv_hi, kv_lo, sb + sw128_offset(4 * vfb + 3, piece), t3);
        }
        if (kc + 1 < chunks) fetch_v((kc + 1) * kChunk);
        // P[row][key]: this thread's 32 keys are span `half` of the chunk
        {
            uint32_t v[32];
            const int col0 = kc * kChunk + half * 32;
            tmem_ld_32x32(t_row + (uint32_t)col0, v);
            tmem_ld_wait();
            float p[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                p[j] = (col0 + j < S) ? exp2f(__uint_as_float(v[j]) - m) : 0.0f;
                l += p[j];
            }
            const uint32_t sb = (uint32_t)(half * kSpanBytesA);
#pragma unroll
            for (int g = 0; g < 8; ++g)
                store_split4(qp_hi, qp_lo, sb + sw128_offset(row, g), make_float4(p[4 * g], p[4 * g + 1], p[4 * g + 2], p[4 * g + 3]));
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            issue_split_mma(tmem_o, tmem_o_corr, smem_u32(qp_hi), smem_u32(qp_lo), kSpanBytesA, smem_u32(kv_hi),
                            smem_u32(kv_lo), kSpanBytesB, kc > 0);
            umma_commit(smem_u32(&mma_bar));
        }
        wait_mma();
    }

    // ---------------- phase 4: ctx = O / row sum
    row_part[half][row] = l;
    __syncthreads();
    if (ok) {  // (uniform: the TMEM load below is a warp-wide instruction, only the stores depend on the row)
        const float inv = 1.0f / (row_part[0][row] + row_part[1][row]);
        uint32_t v[32];
        tmem_ld_32x32(t_row + (uint32_t)(s_pad + half * 32), v);
        tmem_ld_wait();
        if (two_acc) {
            uint32_t w[32];
            tmem_ld_32x32(t_row + (uint32_t)(s_pad + kHeadDim + half * 32), w);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
        }
        const bool row_ok = q0 + row < S;
        const int64_t at = (seq * (int64_t)S + q0 + row) * H + head * kHeadDim + half * 32;
        float y[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = __uint_as_float(v[j]) * inv;
        if (ctx != nullptr && row_ok) {
#pragma unroll
            for (int g = 0; g < 8; ++g)
                *reinterpret_cast<float4 *>(ctx + at + 4 * g) = make_float4(y[4 * g], y[4 * g + 1], y[4 * g + 2], y[4 * g + 3]);
        }
        if (ctx_q != nullptr && row_ok) {  // the same fp32 values, quantised for the next quantised layer (Eq. 1)
            const float Sq = __ldg(S_q);
#pragma unroll
            for (int g = 0; g < 2; ++g)
                *reinterpret_cast<uint4 *>(ctx_q + at + 16 * g) = make_uint4(
                    quantize_pack4(y[16 * g + 0], y[16 * g + 1], y[16 * g + 2], y[16 * g + 3], Sq),
                    quantize_pack4(y[16 * g + 4], y[16 * g + 5], y[16 * g + 6], y[16 * g + 7], Sq),
                    quantize_pack4(y[16 * g + 8], y[16 * g + 9], y[16 * g + 10], y[16 * g + 11], Sq),
                    quantize_pack4(y[16 * g + 12], y[16 * g + 13], y[16 * g + 14], y[16 * g + 15], Sq));
        }
    }

    // ---------------- teardown (reached by every thread, also after a time-out)
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

bool g_attention_tc_enabled = true;

}  // namespace

void set_attention_tensor_cores(bool enable) { g_attention_tc_enabled = enable; }

// Device status word of the tensor-core attention kernel (one per device, in a file-scope array).
static __device__ int32_t g_attention_status[1];

int32_t *attention_status_word()
{
    static int32_t *cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (cached[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_attention_status) != cudaSuccess) return nullptr;
        cached[dev] = static_cast<int32_t *>(p);
    }
    return cached[dev];
}

bool attention_tc_supported(const float *qkv, int64_t S, int64_t heads, const float *ctx, const int8_t *ctx_q)
{
    const int64_t s_pad = (S + kChunk - 1) / kChunk * kChunk;
    auto al16 = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    (void)heads;  // H = 64 * heads keeps every row 16-byte aligned
    return g_attention_tc_enabled && s_pad + kHeadDim <= 512 && al16(qkv) && al16(ctx) && al16(ctx_q);
}

cudaError_t launch_attention_tc(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                                int8_t *ctx_q, cudaStream_t s)
{
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnTcSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int64_t s_pad = (S + kChunk - 1) / kChunk * kChunk;
    uint32_t cols = 32;
    while (cols < (uint32_t)(s_pad + kHeadDim)) cols <<= 1;  // (a second O accumulator is used when 64 more columns fit)
    dim3 grid((unsigned)((S + kQTile - 1) / kQTile), (unsigned)heads, (unsigned)B);
    attention_tc_kernel<<<grid, kThreads, kAttnTcSmemBytes, s>>>(qkv, (int)S, heads * kHeadDim, 1.4426950408889634f / 8.0f,
                                                                 ctx, S_q, ctx_q, cols, attention_status_word());
    return cudaGetLastError();
}

}  // namespace q8
