// Int8 x Int8 -> Int32 GEMM with the fused Q8BERT epilogue on Blackwell tensor cores (sm_100a).
//
// Sec. 3 (inference mode): acc = X_q W_q^T in Int32, accumulated onto the Int32 bias, then
// dequantised by 1 / (S_x S_w) and optionally passed through GELU, all inside one kernel:
//
//   warp 0      TMA producer: 128-byte-swizzled K-major tiles of X_q [M,K] and W_q [N,K] go
//               global -> shared through a ring of mbarrier-guarded stages
//   warp 1      MMA issuer: one lane issues tcgen05.mma kind::i8; Int32 accumulators live in
//               TMEM, double buffered
//   warps 2..9  epilogue: tcgen05.ld the accumulator, add b_q, convert, scale, GELU, stage the
//               fp32 block in swizzled shared memory and write it with a TMA store
//
// Two shapes of the same kernel: CTAS = 1 (one SM per 128 x BLOCK_N tile) for small problems, and
// CTAS = 2 (cta_group::2: a pair of SMs shares one 256 x 256 tile, each loading its own 128 rows
// of X_q and its own half of the W_q rows), which halves the operand bytes each SM must pull from
// L2 per MAC.  No cluster multicast load is used anywhere.
//
// The kernel is persistent (a static tile list per CTA / CTA pair), so the epilogue of tile i
// overlaps the main loop of tile i+1.  Every wait on an mbarrier is bounded: after ~2 s the CTA
// raises Q8_ERR_TIMEOUT in the status word, all roles leave their loops, in-flight copies are
// drained and TMEM is released before the CTA exits.

#include <cuda.h>

#include "q8_gemm_common.cuh"

namespace q8 {

namespace {

using namespace ptx;
using namespace gemm_detail;

constexpr int kAccStages = 2;      // TMEM accumulator double buffering
// Epilogue warps per CTA (template parameter EW): 8 = two per TMEM lane quarter, each taking half of the tile's
// columns; 16 = four per quarter.  A warp walks its 32-column blocks one after the other and every block is a
// chain of dependent latencies (TMEM load, arithmetic, staging, proxy fence, TMA store), so when the main loop is
// short (small K) more warps shorten the epilogue; the extra staging buffers cost one stage of the operand ring.

template <int BLOCK_N, int CTAS, int EW>
struct Cfg {
    static constexpr int kEpilogueWarps = EW;
    static constexpr int kThreads = 96 + 32 * EW;  // two TMA producer warps, the MMA warp, EW epilogue warps
    static constexpr int kBRows = BLOCK_N / CTAS;  // W_q rows each CTA loads
    static constexpr int kABytes = BLOCK_M * BLOCK_K;
    static constexpr int kBBytes = kBRows * BLOCK_K;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStagingBytes = kEpilogueWarps * kStagingBytesPerWarp;
    // b_q of the 32 columns a warp is working on.  With 16 epilogue warps these 2 KB are what stands between four
    // and five stages of the operand ring, so there the exchange happens inside the warp's own staging buffer.
    static constexpr bool kBiasInStaging = EW == 16;
    static constexpr int kBiasBytes = kBiasInStaging ? 0 : kEpilogueWarps * 32 * 4;
    static constexpr int kRingBudget = 227 * 1024 - 1024 - 128 - kStagingBytes - kBiasBytes;  // left for the operand ring
    static constexpr int kStages = kRingBudget / kStageBytes > 8 ? 8 : kRingBudget / kStageBytes;
    static constexpr int kTmemCols = kAccStages * BLOCK_N < 32 ? 32 : kAccStages * BLOCK_N;
    static constexpr int kBarrierBytes = (2 * kStages + 2 * kAccStages) * 8 + 16;
    // +1024: the dynamic shared window is only 16-byte aligned; tiles need 1024 (swizzle atom)
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kStagingBytes + kBiasBytes + kBarrierBytes;
    static constexpr int kColsPerWarp = BLOCK_N / (EW / 4) < 32 ? 32 : BLOCK_N / (EW / 4);  // narrow tiles idle some warps
    static_assert((kTmemCols & (kTmemCols - 1)) == 0 && kTmemCols <= 512, "TMEM columns: power of two <= 512");
    static_assert(BLOCK_N % 32 == 0 && BLOCK_N >= 32 && BLOCK_N <= 256, "UMMA N");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    // Instruction descriptor of tcgen05.mma kind::i8: D = S32, A = B = signed 8-bit, both K-major.
    static constexpr uint32_t kInstrDesc = (2u << 4)                                    // D format: S32
                                           | (1u << 7)                                  // A format: signed int8
                                           | (1u << 10)                                 // B format: signed int8
                                           | ((uint32_t)(BLOCK_N >> 3) << 17)           // N / 8
                                           | ((uint32_t)((BLOCK_M * CTAS) >> 4) << 24); // M / 16
};

// ------------------------------------------------------------------ the kernel
// OUT: what the epilogue writes.  kOutPlain: fp32 Y, staged in shared memory and stored by TMA (or by the lanes
// when Y is not aligned for that); kOutInt8: only the Int8 copy; kOutFull: fp32 and / or Int8 and / or the debug copy
// of the accumulator, as asked for; kOutDirect: fp32 Y stored straight from the accumulator fragments.  Separate
// instantiations, so that a layer does not carry the registers of the paths it does not take.

template <int BLOCK_N, int CTAS, int EW, bool ABSMAX, int OUT>
__global__ void __launch_bounds__(96 + 32 * EW, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    const __grid_constant__ CUtensorMap tmap_w2, const __grid_constant__ CUtensorMap tmap_w4,
                    const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_yq, GemmArgs a,
                    int tma_store, int yq_tma, int64_t full_tiles, int split)
{
    using C = Cfg<BLOCK_N, CTAS, EW>;
    constexpr int kEpilogueWarps = EW;
    constexpr int TILE_M = BLOCK_M * CTAS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *smem_a = smem;
    uint8_t *smem_b = smem + C::kStages * C::kABytes;
    uint8_t *smem_stage = smem + C::kStages * C::kStageBytes;  // multiple of 1024 from the base
    int32_t *smem_bq = reinterpret_cast<int32_t *>(smem_stage + C::kStagingBytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(smem_bq) + C::kBiasBytes);
    uint64_t *full_bar = bars;
    uint64_t *empty_bar = bars + C::kStages;
    uint64_t *tmem_full_bar = bars + 2 * C::kStages;
    uint64_t *tmem_empty_bar = tmem_full_bar + kAccStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tmem_empty_bar + kAccStages);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = CTAS == 2 ? cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;
    const int64_t unit = blockIdx.x / CTAS, num_units = gridDim.x / CTAS;  // a unit = one CTA or one CTA pair
    const int64_t tiles_n = (a.N + BLOCK_N - 1) / BLOCK_N;
    const int64_t tiles_m = (a.M + TILE_M - 1) / TILE_M;
    // Tile schedule.  Tiles [0, full_tiles) are whole BLOCK_N-wide tiles and fill complete rounds over the
    // units; the leftover tiles of the last, partial round are cut into `split` narrower tiles each (same rows,
    // BLOCK_N / split columns), so that the tail keeps more units busy for a shorter time.
    const int64_t num_tiles = full_tiles + (tiles_m * tiles_n - full_tiles) * split;
    const int32_t tiles_n32 = (int32_t)tiles_n, full32 = (int32_t)full_tiles;  // tile counts fit 32 bits by far
    // Every warp decodes a tile index per tile, and in the epilogue warps that sits on the serial path between two
    // accumulators, so it avoids integer division: split is 1, 2 or 4 (a shift), and whole / tiles_n is the high
    // word of whole * ceil(2^32 / tiles_n), exact while whole * tiles_n < 2^32 (else the division is kept).
    const int split_log2 = split >> 1;
    const uint32_t tn_magic = 0xFFFFFFFFu / (uint32_t)tiles_n32 + 1u;
    const bool tn_fast = tiles_n32 > 1 && (uint64_t)(tiles_m * tiles_n) * (uint64_t)tiles_n < (uint64_t(1) << 32);
    auto decode = [&](int64_t t, int64_t &m_idx, int64_t &n0, int &width) {
        int32_t whole = (int32_t)t, sub = 0;
        width = BLOCK_N;
        if (whole >= full32) {
            const int32_t u = whole - full32;
            width = BLOCK_N >> split_log2;
            whole = full32 + (u >> split_log2);
            sub = u & (split - 1);
        }
        const int32_t mi = tn_fast ? (int32_t)__umulhi((uint32_t)whole, tn_magic) : whole / tiles_n32;
        m_idx = mi;
        n0 = (whole - mi * tiles_n32) * BLOCK_N + sub * width;
    };
    const int num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);   // the (leader's) producer arrives once, with the byte count
            mbar_init(smem_u32(empty_bar + s), 1);  // one tcgen05.commit per use
        }
        for (int s = 0; s < kAccStages; ++s) {
            mbar_init(smem_u32(tmem_full_bar + s), 1);
            mbar_init(smem_u32(tmem_empty_bar + s), kEpilogueWarps * CTAS);  // every epilogue warp of the unit
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (CTAS == 2) tmem_alloc_pair(smem_u32(tmem_slot), C::kTmemCols);
        else tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
    }
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();  // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above touched only this CTA's own resources; the kernel before this one in the stream (which
    // produced X_q) must be complete before anything below reads global memory
    grid_dependency_release_next(num_tiles <= 3 * num_units);  // up to three rounds of tiles count as small
    grid_dependency_wait();

    if (warp == 0 || warp == 2) {
        // ---------------- TMA producers (each CTA loads its own rows) ----------------
        // Two warps, each a converged warp with one elected issuing lane (like the MMA warp below): warp 0 takes the
        // even k-blocks of the CTA's sequence of (tile, k-block) steps, warp 2 the odd ones.  One trip of a
        // producer (wake up on the freed stage, arm the barrier, issue two tensor loads) takes 400 to 600 cycles,
        // as long as the tensor cores need for the k-block (4 MMAs of 128 cycles), so a single producer cannot
        // keep the ring full.
        {
            const int p = warp >> 1;  // 0 or 1
            const uint32_t elected = elect_one();
            int s = p % C::kStages;
            uint32_t phase = 0;
            int issued = 0;
            int64_t g = p;  // index of the step in the CTA's sequence (slot g % kStages, parity (g / kStages) & 1)
            bool ok = true;
            int kb = p;
            int64_t tile = unit;
            while (kb >= num_kb && tile < num_tiles) { kb -= num_kb; tile += num_units; }
            while (ok && tile < num_tiles) {
                int64_t m_idx, n_start;
                int width;
                decode(tile, m_idx, n_start, width);
                const int b_rows = width / CTAS;  // W_q rows this CTA loads for the tile
                const int32_t m0 = (int32_t)(m_idx * TILE_M + cta_rank * BLOCK_M);
                const int32_t n0 = (int32_t)(n_start + cta_rank * b_rows);
                const CUtensorMap *map_w = width == BLOCK_N ? &tmap_w : (width * 2 == BLOCK_N ? &tmap_w2 : &tmap_w4);
                const uint32_t stage_bytes = (uint32_t)(C::kABytes + b_rows * BLOCK_K);
                for (; kb < num_kb; kb += 2) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(empty_bar + s), phase ^ 1u, abort_flag, a.status));
                    if (!ok) break;
                    const uint32_t fb = smem_u32(full_bar + s);
                    const uint32_t dst_a = smem_u32(smem_a + s * C::kABytes), dst_b = smem_u32(smem_b + s * C::kBBytes);
                    if (CTAS == 1) {
                        mbar_expect_tx_elected(elected, fb, stage_bytes);
                        tma_load_2d_elected(elected, dst_a, &tmap_x, kb * BLOCK_K, m0, fb);
                        tma_load_2d_elected(elected, dst_b, map_w, kb * BLOCK_K, n0, fb);
                    } else {
                        // both CTAs report their bytes to the leader's barrier, which the MMA warp waits on
                        if (leader) mbar_expect_tx_elected(elected, fb, 2 * stage_bytes);
                        const uint32_t fb_leader = map_to_cta(fb, 0);
                        tma_load_2d_pair_elected(elected, dst_a, &tmap_x, kb * BLOCK_K, m0, fb_leader);
                        tma_load_2d_pair_elected(elected, dst_b, map_w, kb * BLOCK_K, n0, fb_leader);
                    }
                    ++issued;
                    g += 2;
                    s += 2;
                    if (s >= C::kStages) { s -= C::kStages; phase ^= 1u; }
                }
                if (!ok) break;
                do { kb -= num_kb; tile += num_units; } while (kb >= num_kb && tile < num_tiles);
            }
            if (!ok) {
                // Aborting: let this warp's copies already issued land before the CTA gives up its shared memory.
                const uint64_t t0 = global_timer_ns();
                if (CTAS == 1 || leader) {
                    const int mine = (C::kStages + 1) / 2;  // at most this many of a producer's steps are in flight
                    const int pending = issued < mine ? issued : mine;
                    for (int i = 0; i < pending; ++i) {
                        const int64_t k = g - 2 * (i + 1);  // the i-th most recent step of this producer
                        const uint32_t par = (uint32_t)((k / C::kStages) & 1);
                        while (!mbar_try_wait(smem_u32(full_bar + k % C::kStages), par) &&
                               global_timer_ns() - t0 < 50000000ull) {}
                    }
                } else {
                    while (global_timer_ns() - t0 < 1000000ull) {}  // the peer cannot poll the leader's barrier
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (the leader CTA drives the pair) ----------------
        // The warp stays converged: every lane waits and computes the same descriptors (which the compiler can then
        // hold in uniform registers, where tcgen05.mma wants them) and one elected lane issues the tensor-core
        // instructions.  Against a single active lane: FFN2 (K = 4096, issue-rate sensitive) 80.3 -> 77.2 us, the
        // other shapes 0-3 % faster.
        if (leader) {
            const uint32_t elected = elect_one();
            auto uniform = [&](bool mine) { return (bool)__all_sync(0xffffffffu, mine); };
            int s = 0;
            uint32_t phase = 0;
            int as = 0;
            uint32_t aphase = 0;
            bool ok = true, committed = false;
            int last_as = 0;
            uint32_t last_aphase = 0;
            for (int64_t tile = unit; ok && tile < num_tiles; tile += num_units) {
                ok = uniform(mbar_wait(smem_u32(tmem_empty_bar + as), aphase ^ 1u, abort_flag, a.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(as * BLOCK_N);
                // a narrow tile of the split tail runs the same MMA with a smaller N field (bits 17..22 = N / 8)
                const uint32_t width = tile < full_tiles ? (uint32_t)BLOCK_N : (uint32_t)(BLOCK_N >> split_log2);
                const uint32_t idesc = (C::kInstrDesc & ~(0x3Fu << 17)) | ((width >> 3) << 17);
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = uniform(mbar_wait(smem_u32(full_bar + s), phase, abort_flag, a.status));
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t da = smem_desc_sw128(smem_u32(smem_a + s * C::kABytes));
                    const uint64_t db = smem_desc_sw128(smem_u32(smem_b + s * C::kBBytes));
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                        // +32 bytes along K inside the swizzle span == +2 in the (addr >> 4) field
                        const uint64_t adv = (uint64_t)(k * (UMMA_K >> 4));
                        if (CTAS == 2) umma_i8_pair_elected(elected, tmem_d, da + adv, db + adv, idesc, (uint32_t)((kb | k) != 0));
                        else umma_i8_elected(elected, tmem_d, da + adv, db + adv, idesc, (uint32_t)((kb | k) != 0));
                    }
                    // frees the stage (in both CTAs) once these MMAs have read it
                    if (CTAS == 2) umma_commit_pair_elected(elected, smem_u32(empty_bar + s));
                    else umma_commit_elected(elected, smem_u32(empty_bar + s));
                    if (++s == C::kStages) { s = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (CTAS == 2) umma_commit_pair_elected(elected, smem_u32(tmem_full_bar + as));  // accumulator complete
                else umma_commit_elected(elected, smem_u32(tmem_full_bar + as));
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
        const int ew = warp - 3;       // 0 .. EW-1
        const int quarter = warp & 3;  // TMEM lanes this warp may touch: 32*quarter .. +31
        const int col_group = ew >> 2;  // which share of the tile's columns this warp takes
        const float S_x = __ldg(a.S_x);
        // product scale S_x * S_w of the 32-column block starting at column n (w_seg is a multiple of 32 here,
        // so a block never straddles two weight-scale segments)
        auto product_scale = [&](int64_t n) {
            const int64_t seg = (a.w_seg > 0 && n < a.N) ? n / a.w_seg : 0;
            return __fmul_rn(S_x, __ldg(a.S_w + seg));
        };
        uint8_t *stage = smem_stage + ew * kStagingBytesPerWarp;
        // (inside the staging buffer: the first 128 bytes when fp32 blocks are staged, which are free once the
        // previous block's TMA store has read them, or past the 32 x 64 staged Int8 bytes of an Int8-only tile)
        int32_t *bq_s = C::kBiasInStaging ? reinterpret_cast<int32_t *>(stage + (a.Y == nullptr ? 2048 : 0)) : smem_bq + ew * 32;
        int as = 0;
        uint32_t aphase = 0;
        bool ok = true;
        float absmax_run = 0.0f;  // max|y| over everything this lane has stored (only kept when a.y_absmax is given)
        // The bias values of a tile are fetched one tile ahead: under the operand traffic of the main loop a
        // global load takes microseconds, which would otherwise be exposed at the start of every tile.
        constexpr int NCH = C::kColsPerWarp / 32;
        float bias_next[NCH];
        // Columns of a tile of `width` columns are shared out in equal runs of at least 32: warp group g takes
        // [g * cpw, (g + 1) * cpw); on a narrow tile the groups past the end have nothing to do.
        auto cols_per_warp = [&](int width) { return max(32, width / (EW / 4)); };
        auto fetch_bias = [&](int64_t tile, float (&dst)[NCH]) {
            int64_t m_idx, n0;
            int width = BLOCK_N;
            if (tile < num_tiles) decode(tile, m_idx, n0, width);
            else n0 = a.N;
            const int cpw = cols_per_warp(width), col_off = col_group * cpw;
#pragma unroll
            for (int ci = 0; ci < NCH; ++ci) {
                const int64_t n = n0 + col_off + 32 * ci + lane;
                dst[ci] = (col_off < width && 32 * ci < cpw && a.bias != nullptr && n < a.N) ? __ldg(a.bias + n) : 0.0f;
            }
        };
        fetch_bias(unit, bias_next);
        // one weight scale for the whole matrix (the usual case): the product scale and its reciprocal are
        // computed once, not per tile (the load of S_w alone is a round trip to L2 under full operand traffic)
        const bool one_scale = a.w_seg <= 0;
        const float S_out_all = __fmul_rn(S_x, __ldg(a.S_w)), inv_all = __fdiv_rn(1.0f, S_out_all);
        for (int64_t tile = unit; ok && tile < num_tiles; tile += num_units) {
            int64_t m_idx, n0;
            int width;
            decode(tile, m_idx, n0, width);
            const int64_t m0 = m_idx * TILE_M + cta_rank * BLOCK_M;
            const int cpw = cols_per_warp(width), col_off = col_group * cpw;
            const bool active = col_off < width;
            // b_q of this warp's columns (Sec. 3: bias quantised at S_x * S_w)
            int32_t bqv[NCH];
            float invv[NCH];
#pragma unroll
            for (int ci = 0; ci < NCH; ++ci) {
                const float S_out = one_scale ? S_out_all : product_scale(n0 + col_off + 32 * ci);
                bqv[ci] = quantize_bias(bias_next[ci], S_out);
                invv[ci] = one_scale ? inv_all : __fdiv_rn(1.0f, S_out);
            }
            fetch_bias(tile + num_units, bias_next);
            ok = mbar_wait(smem_u32(tmem_full_bar + as), aphase, abort_flag, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            // Hands the accumulator buffer back to the MMA warp (called once this warp's TMEM loads are done:
            // tcgen05.wait::ld has returned in every lane, so the values are in registers).  The arrival carries no
            // memory ordering: nothing this warp wrote to memory is read by the MMA warp.
            auto release = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (CTAS == 2) mbar_arrive_cluster_relaxed(map_to_cta(smem_u32(tmem_empty_bar + as), 0));
                    else mbar_arrive(smem_u32(tmem_empty_bar + as));
                }
            };
            if (active && OUT == kOutDirect)
                epilogue_warp_direct<C::kColsPerWarp, ABSMAX>(
                    a, tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(as * BLOCK_N + col_off),
                    m0 + quarter * 32, n0 + col_off, bqv, invv, bq_s, lane, cpw / 32, release, absmax_run);
            else if (active)
                epilogue_warp<C::kColsPerWarp, ABSMAX, (EW == 8), C::kBiasInStaging, OUT>(a, &tmap_y, tma_store == 1, &tmap_yq, yq_tma != 0,
                                               tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(as * BLOCK_N + col_off),
                                               m0 + quarter * 32, n0 + col_off, bqv, invv, stage, bq_s, lane, cpw / 32, release,
                                               absmax_run);
            else
                release();
            if (++as == kAccStages) { as = 0; aphase ^= 1u; }
        }
        if (ABSMAX) warp_fold_absmax(absmax_run, a.y_absmax);  // one atomic per epilogue warp and launch
        if (lane == 0) tma_store_wait_all();
    }

    // ---------------- teardown (reached by every thread, also when aborting) ----------------
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) {
        __syncwarp();
        cluster_sync_all();  // the peer has finished with this CTA's barriers and with the shared accumulators
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if (CTAS == 2) tmem_dealloc_pair(tmem_base, C::kTmemCols);
        else tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ------------------------------------------------------------------ host side
int g_force_block_n = 0, g_force_ctas = 0;  // set by q8_tune_gemm_tile(); 0 = choose automatically
int g_force_epilogue_warps = 0;            // 0 automatic, else 8 or 16 (cta_group::2 kernel only)
int g_direct_store = -1;                   // fp32-only output stored straight from registers: 1 yes, 0 no, -1 automatic
bool g_tail_split_enabled = true;          // cut the tiles of a partial last round into narrower ones

template <int BLOCK_N, int CTAS, int EW, bool ABSMAX, int OUT>
cudaError_t launch_cfg_impl(const GemmArgs &a, cudaStream_t s);

// Unstaged stores of a plain fp32 output: chosen automatically where they measured faster, i.e. with a long main loop
// (the 8-warp epilogue of the CTA pair, K > 2048: FFN2 75.1 -> 73.7 us, no staging traffic in shared memory, which the
// operand ring and the tensor cores already load fully); with a short one the staged TMA stores win (QKV 79.5
// against 85.7 us).  The pair kernels alone have the instantiation.
template <int CTAS, int EW>
bool wants_direct_store(const GemmArgs &a)
{
    const bool direct = g_direct_store < 0 ? (CTAS == 2 && EW == 8) : g_direct_store != 0;
    return CTAS == 2 && direct && a.Y != nullptr && a.Yq == nullptr && a.dbg_acc == nullptr && ((a.N & 1) == 0) &&
           ((reinterpret_cast<uintptr_t>(a.Y) & 7u) == 0);
}

// The layer that also reports max|y| (Sec. 4.1 chained dynamically) and each output mode run their own
// instantiation of the kernel.
template <int BLOCK_N, int CTAS, int EW, bool ABSMAX>
cudaError_t launch_cfg_out(const GemmArgs &a, cudaStream_t s)
{
    if (a.Yq != nullptr && a.Y == nullptr && a.dbg_acc == nullptr)
        return launch_cfg_impl<BLOCK_N, CTAS, EW, ABSMAX, kOutInt8>(a, s);
    if (a.Yq != nullptr || a.dbg_acc != nullptr) return launch_cfg_impl<BLOCK_N, CTAS, EW, ABSMAX, kOutFull>(a, s);
    if constexpr (CTAS == 2) {
        if (wants_direct_store<CTAS, EW>(a)) return launch_cfg_impl<BLOCK_N, CTAS, EW, ABSMAX, kOutDirect>(a, s);
    }
    return launch_cfg_impl<BLOCK_N, CTAS, EW, ABSMAX, kOutPlain>(a, s);
}
template <int BLOCK_N, int CTAS, int EW = 8>
cudaError_t launch_cfg(const GemmArgs &a, cudaStream_t s)
{
    return a.y_absmax != nullptr ? launch_cfg_out<BLOCK_N, CTAS, EW, true>(a, s)
                                 : launch_cfg_out<BLOCK_N, CTAS, EW, false>(a, s);
}

template <int BLOCK_N, int CTAS, int EW, bool ABSMAX, int OUT>
cudaError_t launch_cfg_impl(const GemmArgs &a, cudaStream_t s)
{
    using C = Cfg<BLOCK_N, CTAS, EW>;
    constexpr int kThreads = C::kThreads;
    auto kernel = gemm_tcgen05_kernel<BLOCK_N, CTAS, EW, ABSMAX, OUT>;
    static bool attr_set[64] = {};  // the opt-in shared-memory size is a per-device, per-function attribute
    static int max_units[64] = {};  // co-resident CTAs (CTAS = 1) or CTA pairs (CTAS = 2) on the device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        if (e != cudaSuccess) return e;
        int units = sm_count() / CTAS;
        if (CTAS == 2) {
            cudaLaunchConfig_t probe = {};
            probe.gridDim = dim3((unsigned)(2 * units));
            probe.blockDim = dim3(kThreads);
            probe.dynamicSmemBytes = C::kSmemBytes;
            cudaLaunchAttribute pattr;
            pattr.id = cudaLaunchAttributeClusterDimension;
            pattr.val.clusterDim.x = 2;
            pattr.val.clusterDim.y = 1;
            pattr.val.clusterDim.z = 1;
            probe.attrs = &pattr;
            probe.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &probe) == cudaSuccess && clusters > 0 &&
                clusters < units)
                units = clusters;
            (void)cudaGetLastError();
        }
        max_units[dev] = units;
        attr_set[dev] = true;
    }
    const int64_t tiles = ((a.M + BLOCK_M * CTAS - 1) / (BLOCK_M * CTAS)) * ((a.N + BLOCK_N - 1) / BLOCK_N);
    const int units = (int)(tiles < max_units[dev] ? tiles : max_units[dev]);
    // Tail of the schedule: when the last round would leave most units idle, its tiles are cut into 2 or 4
    // narrower ones (as many as still fit in one round), so the round is shorter by the saved W traffic and MMAs.
    int split = 1;
    int64_t full_tiles = tiles;
    if (CTAS == 2 && g_tail_split_enabled && tiles > units && tiles % units != 0) {
        const int64_t rest = tiles % units;
        split = rest * 4 <= units ? 4 : (rest * 2 <= units ? 2 : 1);
        if (split > 1) full_tiles = tiles - rest;
    }
    CUtensorMap tx, tw, tw2, tw4, ty;
    if (!make_tmap(&tx, a.Xq, a.M, a.K, BLOCK_M) || !make_tmap(&tw, a.Wq, a.N, a.K, C::kBRows))
        return cudaErrorInvalidValue;
    if (split > 1) {
        if (!make_tmap(&tw2, a.Wq, a.N, a.K, C::kBRows / 2) || !make_tmap(&tw4, a.Wq, a.N, a.K, C::kBRows / 4))
            return cudaErrorInvalidValue;
    } else {
        tw2 = tw;  // never used
        tw4 = tw;
    }
    // the TMA store needs a 16-byte aligned base and row pitch; otherwise lanes store their rows directly
    int tma_store = OUT != kOutDirect && a.Y != nullptr && ((a.N & 3) == 0) &&
                    ((reinterpret_cast<uintptr_t>(a.Y) & 15u) == 0);
    if (tma_store) {
        if (!make_tmap_out(&ty, a.Y, a.M, a.N)) return cudaErrorInvalidValue;
    } else {
        ty = tx;  // never dereferenced
    }
    // Int8-only output (no fp32 Y): full-width tiles leave through TMA stores of the staged Int8 rows
    CUtensorMap tyq = tx;  // never dereferenced unless yq_tma
    constexpr int kCpw = C::kColsPerWarp;
    int yq_tma = (kCpw == 64 || kCpw == 128) && a.Y == nullptr && a.Yq != nullptr && ((a.N & 15) == 0) &&
                 ((reinterpret_cast<uintptr_t>(a.Yq) & 15u) == 0);
    if (yq_tma && !make_tmap_out_q(&tyq, a.Yq, a.M, a.N, kCpw)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * CTAS));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CTAS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // set-up (barriers, TMEM) may overlap the tail of the preceding kernel; see grid_dependency_wait()
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    e = cudaLaunchKernelEx(&cfg, kernel, tx, tw, tw2, tw4, ty, tyq, a, tma_store, yq_tma, full_tiles, split);
    LaunchInfo &li = last_launch_info();
    li.gemm_kernel = 1;
    li.block_n = BLOCK_N;
    li.ctas = CTAS;
    li.epilogue_warps = EW;
    li.grid = units * CTAS;
    li.tail_split = split;
    li.store_mode = OUT == kOutDirect ? 2 : tma_store;
    li.launches += 1;
    return e;
}

// Relative time of one 32-deep K step of a 128 x bn tile on one SM: the tensor pipe needs bn/2 cycles,
// reading the (128 + bn) x 32 operand bytes from shared memory needs (128 + bn)/4; plus a fixed per-step cost.
double tile_step_cost(int bn)
{
    const double mma = bn / 2.0, smem = (128 + bn) / 4.0;
    return (mma > smem ? mma : smem) + 8.0;
}

cudaError_t launch_by_shape(int bn, int ctas, const GemmArgs &a, cudaStream_t s)
{
    if (ctas == 2) {
        // a short main loop (small K) leaves the epilogue on the critical path: give it twice the warps
        const bool wide_epilogue = g_force_epilogue_warps ? g_force_epilogue_warps == 16 : a.K <= 2048;
        return wide_epilogue ? launch_cfg<256, 2, 16>(a, s) : launch_cfg<256, 2, 8>(a, s);
    }
    switch (bn) {
        case 256: return launch_cfg<256, 1>(a, s);
        case 128: return launch_cfg<128, 1>(a, s);
        case 64: return launch_cfg<64, 1>(a, s);
        default: return launch_cfg<32, 1>(a, s);
    }
}

}  // namespace

void set_gemm_tile_override(int block_n, int ctas, int epilogue_warps)
{
    g_force_block_n = block_n;
    g_force_ctas = ctas;
    if (epilogue_warps != 0) g_force_epilogue_warps = epilogue_warps;
}

void set_gemm_tail_split(bool enable) { g_tail_split_enabled = enable; }
void set_gemm_direct_store(int mode) { g_direct_store = mode < 0 ? -1 : (mode != 0); }
void set_gemm_epilogue_warps(int warps) { g_force_epilogue_warps = warps; }

bool tcgen05_gemm_supported(const GemmArgs &a)
{
    return (a.K % 16 == 0) && ((reinterpret_cast<uintptr_t>(a.Xq) & 15u) == 0) &&
           ((reinterpret_cast<uintptr_t>(a.Wq) & 15u) == 0) && a.M < (int64_t(1) << 31) && a.N < (int64_t(1) << 31) &&
           (a.w_seg % 32 == 0);
}

cudaError_t launch_gemm_tcgen05(const GemmArgs &a, cudaStream_t s)
{
    if (g_force_ctas == 2 || (g_force_ctas == 1 && g_force_block_n != 0))
        return launch_by_shape(g_force_block_n, g_force_ctas, a, s);
    const int sms = sm_count();
    // Large problems: CTA pairs on 256 x 256 tiles (least operand traffic per MAC) once every pair has work.
    const int64_t pair_tiles = ((a.M + 255) / 256) * ((a.N + 255) / 256);
    if (a.N >= 192 && a.M > 128 && pair_tiles >= sms / 2) return launch_by_shape(256, 2, a, s);
    // Otherwise single-CTA tiles: pick the width that minimises (waves over the SMs) x (time of one tile).
    const int64_t tm = (a.M + BLOCK_M - 1) / BLOCK_M;
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
    return launch_by_shape(best, 1, a, s);
}

}  // namespace q8
