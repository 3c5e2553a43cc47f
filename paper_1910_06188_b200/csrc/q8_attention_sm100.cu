// Multi-head self-attention (head dimension 64, no mask) on the Blackwell tensor cores with fp32-grade
// accuracy: both products, Q K^T and P V, run as tcgen05.mma kind::tf32 with every fp32 operand split into
// a TF32-exact high part (x rounded to nearest TF32) and the low remainder (x = hi + lo exactly), and
// the three significant partial products hi*hi + hi*lo + lo*hi are accumulated in fp32 in TMEM.  The dropped
// lo*lo term is below 2^-22 relative per product, i.e. at the rounding level of a plain fp32 dot product.
// (The paper keeps attention in fp32 and quantises only the FC layers; this kernel is the fp32 attention an
// encoder forward needs around them.)
//
// One CTA = 128 queries of one (sequence, head): 16 worker warps plus one warp that only issues MMAs.
// All operands are staged by the workers themselves (global -> registers -> split -> shared memory in the
// K-major 128-byte-swizzled layout the MMA reads); no TMA, no multicast.  Chunks of keys go through two (phase 1)
// or three (phase 2) buffer sets, so the MMAs of chunk c run while the workers prepare the chunks after it:
//   phase 1  Q tile (scaled by log2(e)/8) -> Q_hi, Q_lo; per 128 keys: K rows -> K_hi, K_lo; 24 MMAs with N = 128
//            (2 swizzle spans x 4 K steps x 3 partial products) -> scores in TMEM columns [128 c, 128 c + 128); the
//            row maxima are read from TMEM chunk by chunk behind the MMAs (a row is shared by four threads)
//   phase 2  per chunk: p = 2^(s - max) -> P_hi (back into tensor memory over the chunk's scores: the A operand is
//            read from there), P_lo (shared memory; keys along K); V chunk transposed ->
//            [V_hi ; V_lo] stacked as one 128-row B operand, so that one N = 128 MMA yields P_hi V_hi (columns
//            0..63 of the O accumulator) and P_hi V_lo (columns 64..127), and one N = 64 MMA adds P_lo V_hi to the
//            latter: 16 MMAs per chunk.  Keeping the small products in columns of their own also leaves a single
//            rounding per K step on the long accumulation chain.
//   phase 3  (O_main + O_corr) / row sum -> ctx (and optionally Int8 at the next layer's scale)
// The whole score row block lives in TMEM (S_pad + 128 <= 512 columns), so the softmax needs no running
// rescale.  Workers and the MMA warp meet only through mbarriers, and every wait on one is bounded: on a
// time-out the CTA raises Q8_ERR_TIMEOUT in the status word, every role leaves its loops and TMEM is freed.

#include "q8_internal.cuh"
#include "q8_sm100_ptx.cuh"

namespace q8 {

namespace {

using namespace ptx;

constexpr int kHeadDim = 64;
constexpr int kQTile = 128;    // queries per CTA = TMEM lanes
constexpr int kChunk = 64;     // keys per chunk = N of the score MMA = K extent of one P / V chunk
constexpr int kWorkers = 512;  // 16 warps: four per TMEM lane quarter, each taking 16 of a chunk's 64 columns
constexpr int kThreads = kWorkers + 32;        // + the MMA warp
constexpr int kSpanBytesA = kQTile * 128;      // one swizzle span (32 fp32 of K) of a 128-row operand: 16 KB
constexpr int kSpanBytesB = 2 * kChunk * 128;  // ... of the 64-row operand, hi rows then lo rows: 16 KB
constexpr int kLoRowsB = kChunk * 128;         // offset of the lo rows inside a B span
constexpr int kBufQP = 4 * kSpanBytesA;        // {hi, lo} x 2 spans: Q, then P
constexpr int kBufKV = 2 * kSpanBytesB;        // 2 spans x [hi ; lo]: K, then V^T
constexpr int kAttnTcSmemBytes = 1024 + 2 * kBufQP + 2 * kBufKV;  // 193 KB
// Phase 2 needs V^T (hi and lo: kBufKV) and P_lo (half of kBufQP) per chunk: three such sets fill the same 192 KB
// (against two sets: 325.7 -> 322.5 us for 64 x 384 x 16 heads).
constexpr int kSets2 = 3;
constexpr int kSet2Bytes = kBufKV + kBufQP / 2;
static_assert(kSets2 * kSet2Bytes == 2 * kBufQP + 2 * kBufKV, "three phase-2 buffer sets use the whole allocation");
// Phase 1 takes keys 128 at a time (N = 128 score MMAs: half as many instructions, each reading Q once for twice
// the columns).  Its two K buffers of 64 KB ([hi 128 rows | lo 128 rows] per span) lie behind Q; phase 2 reuses the
// whole allocation for its three buffer sets.
constexpr int kBigChunk = 2 * kChunk;
constexpr int kSpanBytesK = 2 * kBigChunk * 128;  // one span of a 128-key K buffer, hi rows then lo rows: 32 KB
constexpr int kLoRowsK = kBigChunk * 128;
static_assert(kBufQP + 2 * (2 * kSpanBytesK) == 2 * kBufQP + 2 * kBufKV, "Q and the two K buffers of phase 1 fill the allocation");

// tcgen05.mma kind::tf32 instruction descriptor: D = F32, A = B = TF32, both K-major, M = 128.
constexpr uint32_t kIdescBase = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kQTile >> 4) << 24);
constexpr uint32_t kIdescN64 = kIdescBase | ((uint32_t)(kChunk >> 3) << 17);         // N = 64
constexpr uint32_t kIdescN128 = kIdescBase | ((uint32_t)((2 * kChunk) >> 3) << 17);  // N = 128

// Byte offset of the 16-byte piece `piece` (0..7) of row `row` inside one swizzle span (rows of 128 bytes,
// groups of 8 rows 1024 bytes apart, piece index XORed with the row's position in its group).
__device__ __forceinline__ uint32_t sw128_offset(int row, int piece)
{
    return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((piece ^ (row & 7)) << 4));
}

// x = hi + lo with hi = x rounded to nearest TF32 (10 explicit mantissa bits, ties away from zero), so
// |lo| <= 2^-12 |x|; lo has up to 12 significant bits, of which the tensor core's truncation of its operands
// keeps 11: an error below 2^-23 |x|.  (Clearing the low bits of x instead would double |lo| and with it that
// error.)  The rounding is done on the integer pipe - add half a TF32 ulp to the bit pattern, clear the 13 low
// bits - which gives what cvt.rna.tf32.f32 gives without loading the conversion unit (22 results per clock and SM).
__device__ __forceinline__ float round_tf32(float x)
{
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}

__device__ __forceinline__ void store_split4(uint8_t *hi_at, uint8_t *lo_at, float4 v)
{
    float4 h;
    h.x = round_tf32(v.x);
    h.y = round_tf32(v.y);
    h.z = round_tf32(v.z);
    h.w = round_tf32(v.w);
    *reinterpret_cast<float4 *>(hi_at) = h;
    *reinterpret_cast<float4 *>(lo_at) = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);  // exact
}

__device__ __forceinline__ void worker_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const float *__restrict__ qkv, int S, int64_t H, float scale, float *__restrict__ ctx,
                    const float *__restrict__ S_q, int8_t *__restrict__ ctx_q, uint32_t *__restrict__ amax,
                    uint32_t tmem_cols, int32_t *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // [ Q, then P buffer 0 | K / V buffer 0 | K / V buffer 1 | P buffer 1 ]
    uint8_t *const q_buf = smem;
    auto k_buf = [&](int b) { return smem + kBufQP + b * (2 * kSpanBytesK); };  // phase 1: two buffers behind Q
    auto v_buf = [&](int b) { return smem + b * kSet2Bytes; };                  // phase 2: three sets of [V^T | P_lo]
    auto plo_buf = [&](int b) { return smem + b * kSet2Bytes + kBufKV; };
    __shared__ __align__(8) uint64_t ready_bar[kSets2];  // workers -> MMA warp: the operands of a chunk are in place
    __shared__ __align__(8) uint64_t done_bar[kSets2];   // MMA warp -> workers: the MMAs of a chunk have completed
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float row_part[4][kQTile];  // per-row partial maxima, then partial sums, of the four column quarters

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q0 = blockIdx.x * kQTile;
    const int64_t head = blockIdx.y, seq = blockIdx.z;
    const int64_t row_pitch = 3 * H;
    const float *base = qkv + seq * (int64_t)S * row_pitch + head * kHeadDim;
    const int chunks = (S + kChunk - 1) / kChunk;
    const int s_pad = chunks * kChunk;
    const int big_chunks = (S + kBigChunk - 1) / kBigChunk;

    if (tid == 0) {
        for (int b = 0; b < kSets2; ++b) {
            mbar_init(smem_u32(&ready_bar[b]), kWorkers / 32);  // one arrival per worker warp
            mbar_init(smem_u32(&done_bar[b]), 1);
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kWorkers / 32) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tmem_o = tmem_base + (uint32_t)s_pad;  // O_main: 64 columns behind the scores; O_corr: the next 64
    grid_dependency_release_next(gridDim.x * gridDim.y * gridDim.z <= 600u);  // up to ~4 waves of CTAs count as small
    grid_dependency_wait();  // the set-up above may overlap the tail of the kernel that produced qkv

    if (warp == kWorkers / 32) {
        // ================= MMA warp: stays converged (all lanes wait and compute the same descriptors, which the
        // compiler can then keep in uniform registers); one elected lane issues, chunk after chunk, as the workers
        // report operands ready
        {
            const uint32_t elected = elect_one();
            uint32_t ready_phase = 0u;  // bit b: parity of the next phase of ready_bar[b]
            bool ok = true;
            const uint32_t q_hi = smem_u32(q_buf), q_lo = q_hi + 2 * kSpanBytesA;
            for (int kc = 0; kc < big_chunks && ok; ++kc) {  // scores of the 128 keys of big chunk kc
                const int b = kc & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&ready_bar[b]), (ready_phase >> b) & 1u, &abort_flag, status));
                ready_phase ^= 1u << b;
                if (!ok) break;
                tc_fence_after();
                const uint32_t d = tmem_base + (uint32_t)(kc * kBigChunk), kb = smem_u32(k_buf(b));
                uint32_t acc = 0u;
#pragma unroll
                for (int span = 0; span < 2; ++span) {
                    const uint64_t ah = smem_desc_sw128(q_hi + span * kSpanBytesA), al = smem_desc_sw128(q_lo + span * kSpanBytesA);
                    const uint64_t bh = smem_desc_sw128(kb + span * kSpanBytesK), bl = smem_desc_sw128(kb + span * kSpanBytesK + kLoRowsK);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {  // 8 fp32 = 32 bytes of K per instruction: +2 in the (address >> 4) field
                        const uint64_t adv = (uint64_t)(2 * ks);
                        umma_tf32_elected(elected, d, al + adv, bh + adv, kIdescN128, acc);  // small terms first
                        umma_tf32_elected(elected, d, ah + adv, bl + adv, kIdescN128, 1u);
                        umma_tf32_elected(elected, d, ah + adv, bh + adv, kIdescN128, 1u);
                        acc = 1u;
                    }
                }
                umma_commit_elected(elected, smem_u32(&done_bar[b]));
            }
            for (int kc = 0, b = 0; kc < chunks && ok; ++kc, b = (b + 1 == kSets2 ? 0 : b + 1)) {  // O += P V of chunk kc
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&ready_bar[b]), (ready_phase >> b) & 1u, &abort_flag, status));
                ready_phase ^= 1u << b;
                if (!ok) break;
                tc_fence_after();
                // P_hi is read from tensor memory, where it has replaced the chunk's scores (row = lane, key = column)
                const uint32_t p_hi = tmem_base + (uint32_t)(kc * kChunk);
                const uint32_t p_lo = smem_u32(plo_buf(b)), vb = smem_u32(v_buf(b));
                uint32_t acc = kc > 0 ? 1u : 0u;
#pragma unroll
                for (int span = 0; span < 2; ++span) {
                    const uint64_t al = smem_desc_sw128(p_lo + span * kSpanBytesA);
                    const uint64_t bhl = smem_desc_sw128(vb + span * kSpanBytesB);  // 128 rows: V_hi then V_lo
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {  // 8 keys per instruction: 8 TMEM columns of P_hi, +2 in the (address >> 4) field
                        const uint64_t adv = (uint64_t)(2 * ks);
                        umma_tf32_ts_elected(elected, tmem_o, p_hi + (uint32_t)(32 * span + 8 * ks), bhl + adv, kIdescN128, acc);  // [P_hi V_hi | P_hi V_lo]
                        umma_tf32_elected(elected, tmem_o + kHeadDim, al + adv, bhl + adv, kIdescN64, 1u);  // += P_lo V_hi
                        acc = 1u;
                    }
                }
                umma_commit_elected(elected, smem_u32(&done_bar[b]));
            }
        }
    } else {
        // ================= workers
        const int quarter = warp & 3, cq = warp >> 2;  // TMEM lane quarter this warp may read; its 16 columns of a chunk
        const int row = quarter * 32 + lane;           // query row (TMEM lane) of this thread in the softmax
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
        uint32_t done_phase = 0u;  // bit b: parity of the next phase of done_bar[b]
        bool ok = true;
        // waits (whole warp, same outcome in every lane) until the MMAs of the chunk that used buffer set b are done
        auto wait_done = [&](int b) {
            const bool mine = mbar_wait(smem_u32(&done_bar[b]), (done_phase >> b) & 1u, &abort_flag, status);
            done_phase ^= 1u << b;
            ok = __all_sync(0xffffffffu, mine);
            tc_fence_after();
        };
        // every thread makes its shared-memory writes visible to the tensor core; then one lane reports for the warp
        // (16 arrivals on the barrier instead of 512)
        auto report_ready = [&](int b) {
            fence_proxy_async_smem();
            tc_fence_before();  // (a tcgen05.st of P_hi has completed by now: tmem_st_wait() before this call)
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ready_bar[b]));
        };

        // ---------------- phase 1: scores = (Q * log2(e)/8) K^T
        constexpr int kPiecesK = (kBigChunk * 16) / kWorkers;  // 16-byte pieces of a 128-key K chunk per thread
        float4 kreg[kPiecesK];
        auto fetch_k = [&](int j0) {  // 128 keys x 64 fp32
#pragma unroll
            for (int i = 0; i < kPiecesK; ++i) {
                const int c = tid + i * kWorkers, r = c >> 4, pc = c & 15;
                kreg[i] = (j0 + r < S) ? __ldg(reinterpret_cast<const float4 *>(base + (int64_t)(j0 + r) * row_pitch + H) + pc)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        };
        fetch_k(0);  // the first K chunk travels while Q is split and staged
        // a 16-byte piece c of a [rows x 64] fp32 tile: row c / 16, span (c % 16) / 8, piece (c % 16) % 8
#pragma unroll
        for (int i = 0; i < (kQTile * 16) / kWorkers; ++i) {
            const int c = tid + i * kWorkers, r = c >> 4, pc = c & 15;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (q0 + r < S) v = __ldg(reinterpret_cast<const float4 *>(base + (int64_t)(q0 + r) * row_pitch) + pc);
            v.x *= scale;
            v.y *= scale;
            v.z *= scale;
            v.w *= scale;
            uint8_t *at = q_buf + (pc >> 3) * kSpanBytesA + sw128_offset(r, pc & 7);
            store_split4(at, at + 2 * kSpanBytesA, v);
        }
        float m = -INFINITY;
        uint32_t sv[32];  // this thread's 32 score columns of a big chunk, on their way out of TMEM
        auto load_scores = [&](int c) { tmem_ld_32x32(t_row + (uint32_t)(c * kBigChunk + cq * 32), sv); };
        auto take_max = [&](int c) {  // after load_scores(c): waits for the load, folds the 32 columns into m
            uint32_t(&v)[32] = sv;
            const int col0 = c * kBigChunk + cq * 32;
            tmem_ld_wait();
            if (col0 + 32 <= S) {
#pragma unroll
                for (int j = 0; j < 32; ++j) m = fmaxf(m, __uint_as_float(v[j]));
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < S) m = fmaxf(m, __uint_as_float(v[j]));
            }
        };
        for (int kc = 0; kc < big_chunks && ok; ++kc) {
            const int b = kc & 1;
            if (kc >= 2) {  // buffer b was read by the MMAs of big chunk kc - 2, whose scores are final after this wait
                wait_done(b);
                if (!ok) break;
                load_scores(kc - 2);  // in flight while the next K chunk is staged below
            }
#pragma unroll
            for (int i = 0; i < kPiecesK; ++i) {
                const int c = tid + i * kWorkers, r = c >> 4, pc = c & 15;
                uint8_t *at = k_buf(b) + (pc >> 3) * kSpanBytesK + sw128_offset(r, pc & 7);
                store_split4(at, at + kLoRowsK, kreg[i]);
            }
            if (kc + 1 < big_chunks) fetch_k((kc + 1) * kBigChunk);  // next K chunk, in flight during the MMAs
            report_ready(b);
            if (kc >= 2) take_max(kc - 2);
        }
        for (int c = (big_chunks > 2 ? big_chunks - 2 : 0); c < big_chunks && ok; ++c) {  // the last two big chunks
            wait_done(c & 1);
            if (ok) {
                load_scores(c);
                take_max(c);
            }
        }
        row_part[cq][row] = m;
        worker_barrier();
        m = fmaxf(fmaxf(row_part[0][row], row_part[1][row]), fmaxf(row_part[2][row], row_part[3][row]));
        worker_barrier();  // row_part is reused for the sums; every score MMA has completed: Q may be overwritten

        // ---------------- phase 2: P = 2^(scores - max), O = P V, chunk by chunk
        float l = 0.0f;
        // V chunk as a 64 x 64 tile of blocks of 4 keys x 2 features: thread = (key block vkb, feature pair vfp); the
        // block is transposed in registers so that each feature row of V^T gets 4 consecutive keys (one 16-byte piece)
        const int vkb = tid >> 5, vfp = tid & 31;
        float2 vreg[4];
        auto fetch_v = [&](int j0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = j0 + 4 * vkb + i;
                vreg[i] = (j < S) ? __ldg(reinterpret_cast<const float2 *>(base + (int64_t)j * row_pitch + 2 * H) + vfp)
                                  : make_float2(0.f, 0.f);
            }
        };
        if (ok) fetch_v(0);
        // All scores are final, so a chunk's 16 score columns are fetched from TMEM one chunk ahead, and its
        // exponentials are taken before the wait for the buffer set they will be stored into.
        uint32_t pv[16];
        if (ok) tmem_ld_32x16(t_row + (uint32_t)(cq * 16), pv);
        for (int kc = 0, b = 0; kc < chunks && ok; ++kc, b = (b + 1 == kSets2 ? 0 : b + 1)) {
            // p = hi + lo (hi = p rounded to TF32).  The hi parts go back into tensor memory over the chunk's scores, from
            // where the MMA takes them as its A operand (no trip through shared memory: 64 x 384 x 16 heads 338 -> 325 us;
            // the same for Q in phase 1 measured slower, 360 us, and is not done); the lo parts go to shared memory.
            float p_lo[16];
            {
                const int col0 = kc * kChunk + cq * 16;
                tmem_ld_wait();
                const bool whole = col0 + 16 <= S;
                uint32_t ph[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    float e;
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(__uint_as_float(pv[j]) - m));
                    const float pj = (whole || col0 + j < S) ? e : 0.0f;
                    l += pj;
                    const float h = round_tf32(pj);
                    ph[j] = __float_as_uint(h);
                    p_lo[j] = pj - h;  // exact
                }
                if (kc + 1 < chunks) tmem_ld_32x16(t_row + (uint32_t)(col0 + kChunk), pv);
                tmem_st_32x16(t_row + (uint32_t)col0, ph);
            }
            if (kc >= kSets2) {  // buffer set b was last read by the MMAs of chunk kc - 3
                wait_done(b);
                if (!ok) break;
            }
            // V^T[d][key]: rows = features (64, hi block then lo block), K = keys of this chunk (2 spans of 32)
            {
                uint8_t *sb = v_buf(b) + (vkb >> 3) * kSpanBytesB;  // keys 4 vkb .. 4 vkb + 3: span vkb / 8, piece vkb % 8
                uint8_t *a0 = sb + sw128_offset(2 * vfp + 0, vkb & 7), *a1 = sb + sw128_offset(2 * vfp + 1, vkb & 7);
                store_split4(a0, a0 + kLoRowsB, make_float4(vreg[0].x, vreg[1].x, vreg[2].x, vreg[3].x));
                store_split4(a1, a1 + kLoRowsB, make_float4(vreg[0].y, vreg[1].y, vreg[2].y, vreg[3].y));
            }
            if (kc + 1 < chunks) fetch_v((kc + 1) * kChunk);
            // P_lo[row][key]: this thread's 16 keys are pieces 4 (cq & 1) .. + 3 of span cq / 2 of the chunk
            {
                uint8_t *sb = plo_buf(b) + (cq >> 1) * kSpanBytesA;
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    *reinterpret_cast<float4 *>(sb + sw128_offset(row, 4 * (cq & 1) + g)) =
                        make_float4(p_lo[4 * g], p_lo[4 * g + 1], p_lo[4 * g + 2], p_lo[4 * g + 3]);
            }
            tmem_st_wait();
            report_ready(b);
        }
        tmem_ld_wait();  // (a load is still in flight only when the loop above was left early)
        row_part[cq][row] = l;  // the row sums are exchanged while the last MMAs run
        worker_barrier();
        for (int c = (chunks > kSets2 ? chunks - kSets2 : 0); c < chunks && ok; ++c) wait_done(c % kSets2);  // the last three chunks

        // ---------------- phase 3: ctx = (O_main + O_corr) / row sum
        if (ok) {  // (warp-uniform: the TMEM loads below are warp-wide instructions, only the stores depend on the row)
            const float inv = 1.0f / ((row_part[0][row] + row_part[1][row]) + (row_part[2][row] + row_part[3][row]));
            uint32_t v[16], w[16];
            tmem_ld_32x16(t_row + (uint32_t)(s_pad + cq * 16), v);
            tmem_ld_32x16(t_row + (uint32_t)(s_pad + kHeadDim + cq * 16), w);
            tmem_ld_wait();
            const bool row_ok = q0 + row < S;
            const int64_t at = (seq * (int64_t)S + q0 + row) * H + head * kHeadDim + cq * 16;
            float y[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) y[j] = (__uint_as_float(v[j]) + __uint_as_float(w[j])) * inv;
            if (amax != nullptr) {  // max|ctx| for a dynamically quantised consumer (Sec. 4.1); rows past S do not count
                float am = 0.0f;
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) am = fmaxf(am, fabsf(y[j]));
                }
                warp_fold_absmax(am, amax);
            }
            if (ctx != nullptr && row_ok) {
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    *reinterpret_cast<float4 *>(ctx + at + 4 * g) = make_float4(y[4 * g], y[4 * g + 1], y[4 * g + 2], y[4 * g + 3]);
            }
            if (ctx_q != nullptr && row_ok) {  // the same fp32 values, quantised for the next quantised layer (Eq. 1)
                const float Sq = __ldg(S_q);
                *reinterpret_cast<uint4 *>(ctx_q + at) =
                    make_uint4(quantize_pack4(y[0], y[1], y[2], y[3], Sq), quantize_pack4(y[4], y[5], y[6], y[7], Sq),
                               quantize_pack4(y[8], y[9], y[10], y[11], Sq), quantize_pack4(y[12], y[13], y[14], y[15], Sq));
            }
        }
    }

    // ---------------- teardown (reached by every thread, also after a time-out)
    tc_fence_before();
    __syncthreads();
    if (warp == kWorkers / 32) {
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
    return g_attention_tc_enabled && s_pad + 2 * kHeadDim <= 512 && al16(qkv) && al16(ctx) && al16(ctx_q);
}

cudaError_t launch_attention_tc(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                                int8_t *ctx_q, uint32_t *amax, cudaStream_t s)
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
    while (cols < (uint32_t)(s_pad + 2 * kHeadDim)) cols <<= 1;  // scores, O_main, O_corr
    dim3 grid((unsigned)((S + kQTile - 1) / kQTile), (unsigned)heads, (unsigned)B);
    const float scale = 1.4426950408889634f / 8.0f;  // log2(e) / sqrt(64): the softmax then uses 2^x
    return launch_overlapping_tail(attention_tc_kernel, grid, dim3(kThreads), kAttnTcSmemBytes, s, qkv, (int)S,
                                   heads * kHeadDim, scale, ctx, S_q, ctx_q, amax, cols, attention_status_word());
}

}  // namespace q8
