// Pieces shared by the tensor-core GEMM kernels of the library: the fused epilogue of one warp (Int32 bias add,
// dequantise, GELU, optional re-quantisation, staged TMA store), its GELU evaluation, and the host-side tensor-map
// construction with a small per-thread cache.
#pragma once

#include <cuda.h>

#include "q8_internal.cuh"
#include "q8_sm100_ptx.cuh"

namespace q8 {
namespace gemm_detail {

using namespace ptx;

constexpr int BLOCK_M = 128;       // accumulator rows per CTA: row i <-> TMEM lane i
constexpr int BLOCK_K = 128;       // bytes == int8 elements per stage row: one 128-byte swizzle span
constexpr int UMMA_K = 32;         // K of one kind::i8 instruction
constexpr int kStagingBytesPerWarp = 32 * 32 * 4;  // the 32 x 32 fp32 block one tcgen05.ld hands to a warp

// ---- GELU without erff, two values at a time: gelu(y) = max(y, 0) - a * Phi(-a), a = |y|, with
// Phi(-a) = 2^p(a) and p a degree-6 fit of log2 Phi(-a) on [0, 5.6] (p(0) = -1 exactly; beyond 5.6
// a * Phi(-a) < 1e-7 and a is clamped).  Absolute error of a * Phi(-a) below 1e-7, so the result is
// within fp32 rounding of the erf form.  The polynomial runs on packed fp32 FMAs (two values per
// instruction, each half rounded like a scalar fmaf) in n = -a = max(-|y|, -5.6), i.e. with the odd
// coefficients negated, so the last step needs no negation: gelu = n * 2^p + max(y, 0).
// Per value: three packed FMA-pipe instructions and a half, one ex2, two min/max.
__device__ __forceinline__ void gelu_fast_x2(uint64_t y2, float &out_lo, float &out_hi)
{
    float y0, y1;
    unpack_f32x2(y2, y0, y1);
    const uint64_t n = pack_f32x2(fmaxf(-fabsf(y0), -5.6f), fmaxf(-fabsf(y1), -5.6f));
    uint64_t p = pack_f32x2(2.9923698093625717e-05f, 2.9923698093625717e-05f);
    p = fma_f32x2(p, n, pack_f32x2(0.0007398707093670964f, 0.0007398707093670964f));
    p = fma_f32x2(p, n, pack_f32x2(0.007977453991770744f, 0.007977453991770744f));
    p = fma_f32x2(p, n, pack_f32x2(0.05323817580938339f, 0.05323817580938339f));
    p = fma_f32x2(p, n, pack_f32x2(-0.45891568064689636f, -0.45891568064689636f));
    p = fma_f32x2(p, n, pack_f32x2(1.1511471271514893f, 1.1511471271514893f));
    p = fma_f32x2(p, n, pack_f32x2(-1.0f, -1.0f));
    float p0, p1, e0, e1;
    unpack_f32x2(p, p0, p1);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(p0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(p1));
    const uint64_t r = fma_f32x2(n, pack_f32x2(e0, e1), pack_f32x2(fmaxf(y0, 0.0f), fmaxf(y1, 0.0f)));
    unpack_f32x2(r, out_lo, out_hi);
}

// ------------------------------------------------------------------ epilogue of one warp
// The warp owns 32 accumulator rows (its TMEM lane quarter) x COLS columns of the tile and walks
// them in 32-column blocks: tcgen05.ld (one row per lane) -> + b_q -> int-to-float ->
// * 1/(S_x S_w) -> GELU -> store.  With tma_store (N % 4 == 0, Y 16-byte aligned) the 32 x 32 fp32
// block is staged in shared memory in the 128-byte-swizzled layout of the output tensor map
// (row = lane, 16-byte piece g at position g ^ (lane & 7): bank-conflict free) and written by one
// TMA store, clipped at the matrix edge by the hardware; otherwise every lane stores its own row.
// Once the last TMEM load of the tile has landed the accumulator buffer is handed back (release()).
// ABSMAX: also keep the running max|y| of what is stored (a compile-time switch, so that the ordinary layer carries
// neither the extra register nor the branch).
// PREFETCH: issue the next block's TMEM load before the proxy fence and TMA store of the current one (pays when a
// warp walks four blocks per tile; with two blocks per warp it measured 1 % slower).
// BIAS_IN_STAGE: bq_s points into `stage`, so a staged fp32 block must have been read by its TMA store before the
// next block's bias values are exchanged there.
// OUT: which outputs the instantiation can write.  kOutPlain: the fp32 Y only; kOutInt8: the Int8 copy only (the
// fused FFN1 of a forward whose next layer is quantised); kOutFull: whatever the call asks for (fp32, Int8, the
// debug copy of the accumulator).  Compiling the other paths out keeps the 16-warp kernel (96 registers per thread)
// free of spills; a spilled value is reloaded from local memory in every block, and under the main loop's traffic
// that load is not a cache hit.
constexpr int kOutPlain = 0, kOutFull = 1, kOutDirect = 2, kOutInt8 = 3;
template <int COLS, bool ABSMAX, bool PREFETCH, bool BIAS_IN_STAGE, int OUT, typename Release>
__device__ __forceinline__ void epilogue_warp(const GemmArgs &a, const CUtensorMap *tmap_y, bool tma_store,
                                              const CUtensorMap *tmap_yq, bool yq_tma, uint32_t taddr, int64_t row0,
                                              int64_t col0, const int32_t (&bqv)[COLS / 32], const float (&invv)[COLS / 32],
                                              uint8_t *stage, int32_t *bq_s, int lane, int nch, Release release,
                                              float &absmax_run)
{
    constexpr int NCHUNK = COLS / 32;  // compile-time maximum; this tile has nch <= NCHUNK blocks (warp-uniform)
    const int64_t row = row0 + lane;
    const bool row_ok = row < a.M;
    constexpr bool kHasY = OUT != kOutInt8, kHasYq = OUT == kOutFull || OUT == kOutInt8, kHasDbg = OUT == kOutFull;
    const float S_y = (kHasYq && a.Yq != nullptr) ? __ldg(a.S_y) : 1.0f;
    const bool yq_vec = ((a.N & 15) == 0) && ((reinterpret_cast<uintptr_t>(a.Yq) & 15u) == 0);
    // Int8-only output of a full-width tile: the warp's 32 x COLS bytes are collected in its staging buffer (free,
    // since no fp32 block is staged) in the swizzled layout of the Int8 output tensor map and leave as one TMA
    // store of whole 64- or 128-byte row pieces instead of 32 separate 16-byte stores per lane and block.
    constexpr bool kYqStageable = COLS == 64 || COLS == 128;
    const bool yq_staged = kHasYq && kYqStageable && yq_tma && nch == NCHUNK;
    const int yq_xor = COLS == 128 ? (lane & 7) : ((lane >> 1) & 3);  // 128-byte / 64-byte swizzle of row `lane`
    bool yq_pending = false;

    // Everything after the TMEM load, for the 32-column block ci held in v, up to and including the staging of the
    // fp32 block in shared memory.  Returns the first column of the block when a staged fp32 block now waits for its
    // proxy fence and TMA store (issue_store below), -1 otherwise; v is dead when it returns.
    auto finish_block = [&](uint32_t (&v)[32], int ci) -> int64_t {
        const int64_t nb = col0 + 32 * ci;
        const float inv = invv[ci];
        if (nb >= a.N || row0 >= a.M) return -1;  // warp-uniform: the block lies outside the matrix
        if (BIAS_IN_STAGE && tma_store && lane == 0) tma_store_wait_read();
        // b_q of these 32 columns (one per lane, computed before the accumulator was ready) -> all lanes
        __syncwarp();
        bq_s[lane] = bqv[ci];
        __syncwarp();
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const int4 b = *reinterpret_cast<const int4 *>(bq_s + 4 * g);
            v[4 * g + 0] = (uint32_t)add_wrap((int32_t)v[4 * g + 0], b.x);
            v[4 * g + 1] = (uint32_t)add_wrap((int32_t)v[4 * g + 1], b.y);
            v[4 * g + 2] = (uint32_t)add_wrap((int32_t)v[4 * g + 2], b.z);
            v[4 * g + 3] = (uint32_t)add_wrap((int32_t)v[4 * g + 3], b.w);
        }
        if (kHasDbg && a.dbg_acc != nullptr && row_ok) {
            int32_t *drow = a.dbg_acc + row * a.N + nb;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (nb + j < a.N) drow[j] = (int32_t)v[j];
        }
        if (a.act == Q8_ACT_GELU) {
            const uint64_t inv2 = pack_f32x2(inv, inv);
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                const uint64_t y2 =
                    mul_f32x2(pack_f32x2(__int2float_rn((int32_t)v[j]), __int2float_rn((int32_t)v[j + 1])), inv2);
                float g0, g1;
                gelu_fast_x2(y2, g0, g1);
                v[j] = __float_as_uint(g0);
                v[j + 1] = __float_as_uint(g1);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__fmul_rn(__int2float_rn((int32_t)v[j]), inv));
        }
        if (ABSMAX && row_ok) {
            // running max|y| of this lane over the outputs that exist (Sec. 4.1: the consumer's dynamic scale)
            const bool whole = nb + 32 <= a.N;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (whole || nb + j < a.N) absmax_run = fmaxf(absmax_run, fabsf(__uint_as_float(v[j])));
        }
        if (kHasYq && a.Yq != nullptr && row_ok) {
            // re-quantised output for the next quantised layer: Eq. 1 at that layer's activation scale
            int8_t *qrow = a.Yq + row * a.N + nb;
            if (yq_staged) {
                // handled below, for all rows of the warp (rows past M are clipped by the store)
            } else if (yq_vec) {  // N % 16 == 0: a 16-byte piece is never split by the edge
                if (nb < a.N)
                    *reinterpret_cast<uint4 *>(qrow) = make_uint4(
                        quantize_pack4(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]), S_y),
                        quantize_pack4(__uint_as_float(v[4]), __uint_as_float(v[5]), __uint_as_float(v[6]), __uint_as_float(v[7]), S_y),
                        quantize_pack4(__uint_as_float(v[8]), __uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]), S_y),
                        quantize_pack4(__uint_as_float(v[12]), __uint_as_float(v[13]), __uint_as_float(v[14]), __uint_as_float(v[15]), S_y));
                if (nb + 16 < a.N)
                    *reinterpret_cast<uint4 *>(qrow + 16) = make_uint4(
                        quantize_pack4(__uint_as_float(v[16]), __uint_as_float(v[17]), __uint_as_float(v[18]), __uint_as_float(v[19]), S_y),
                        quantize_pack4(__uint_as_float(v[20]), __uint_as_float(v[21]), __uint_as_float(v[22]), __uint_as_float(v[23]), S_y),
                        quantize_pack4(__uint_as_float(v[24]), __uint_as_float(v[25]), __uint_as_float(v[26]), __uint_as_float(v[27]), S_y),
                        quantize_pack4(__uint_as_float(v[28]), __uint_as_float(v[29]), __uint_as_float(v[30]), __uint_as_float(v[31]), S_y));
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (nb + j < a.N) qrow[j] = (int8_t)quantize_value(__uint_as_float(v[j]), S_y);
            }
        }
        if (kHasYq && yq_staged) {
            if (!yq_pending) {
                if (lane == 0) tma_store_wait_read();  // the previous tile has left the staging buffer
                __syncwarp();
                yq_pending = true;
            }
            uint8_t *srow = stage + lane * COLS;
            *reinterpret_cast<uint4 *>(srow + (((2 * ci) ^ yq_xor) << 4)) = make_uint4(
                quantize_pack4(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]), S_y),
                quantize_pack4(__uint_as_float(v[4]), __uint_as_float(v[5]), __uint_as_float(v[6]), __uint_as_float(v[7]), S_y),
                quantize_pack4(__uint_as_float(v[8]), __uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]), S_y),
                quantize_pack4(__uint_as_float(v[12]), __uint_as_float(v[13]), __uint_as_float(v[14]), __uint_as_float(v[15]), S_y));
            *reinterpret_cast<uint4 *>(srow + (((2 * ci + 1) ^ yq_xor) << 4)) = make_uint4(
                quantize_pack4(__uint_as_float(v[16]), __uint_as_float(v[17]), __uint_as_float(v[18]), __uint_as_float(v[19]), S_y),
                quantize_pack4(__uint_as_float(v[20]), __uint_as_float(v[21]), __uint_as_float(v[22]), __uint_as_float(v[23]), S_y),
                quantize_pack4(__uint_as_float(v[24]), __uint_as_float(v[25]), __uint_as_float(v[26]), __uint_as_float(v[27]), S_y),
                quantize_pack4(__uint_as_float(v[28]), __uint_as_float(v[29]), __uint_as_float(v[30]), __uint_as_float(v[31]), S_y));
        }
        if (!kHasY || a.Y == nullptr) return -1;
        if (tma_store) {
            if (!BIAS_IN_STAGE && lane == 0) tma_store_wait_read();  // the previous block has left the staging buffer
            __syncwarp();  // (also: every lane has read the bias values before the block overwrites them)
            uint8_t *srow = stage + lane * 128;
#pragma unroll
            for (int g = 0; g < 8; ++g)
                *reinterpret_cast<uint4 *>(srow + ((g ^ (lane & 7)) << 4)) =
                    make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
            return nb;
        } else if (row_ok) {
            float *yrow = a.Y + row * a.N + nb;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (nb + j < a.N) yrow[j] = __uint_as_float(v[j]);
        }
        return -1;
    };
    auto issue_store = [&](int64_t nb) {
        fence_proxy_async_smem();  // generic-proxy writes of the staging -> visible to the TMA (async proxy)
        __syncwarp();
        if (lane == 0) tma_store_2d(tmap_y, (int32_t)nb, (int32_t)row0, smem_u32(stage));
    };

    // With PREFETCH the next block's TMEM load is issued as soon as this block's values have left the registers
    // (staged in shared memory), so its latency runs under the proxy fence and the TMA store of this block.  Either
    // way the accumulator buffer is handed back once the last load of the tile has landed.
    uint32_t v[32];
    if (PREFETCH && nch > 0) tmem_ld_32x32(taddr, v);
#pragma unroll
    for (int ci = 0; ci < NCHUNK; ++ci) {
        if (ci >= nch) break;
        if (!PREFETCH) tmem_ld_32x32(taddr + (uint32_t)(32 * ci), v);
        tmem_ld_wait();
        if (ci + 1 == nch) release();
        const int64_t staged_at = finish_block(v, ci);
        if (PREFETCH && ci + 1 < nch) tmem_ld_32x32(taddr + (uint32_t)(32 * (ci + 1)), v);
        if (staged_at >= 0) issue_store(staged_at);
    }
    if (kHasYq && yq_pending) {
        // blocks beyond column N were never staged; the store clips them (and rows past M) at the matrix edge
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) tma_store_2d(tmap_yq, (int32_t)col0, (int32_t)row0, smem_u32(stage));
    }
}

// The same work for the plain fp32 output (no Int8 copy), without the shared-memory staging: the accumulator block is
// read in the 16x256b fragment layout, where four neighbouring lanes hold 32 contiguous bytes of a row, so each lane
// stores its pairs straight to Y (8-byte stores, every sector written whole by one instruction).  No proxy fence,
// no TMA store, no staging buffer to wait for.  Needs an even N and an 8-byte aligned Y; like the plain form of the
// staged epilogue it writes Y only (a call that wants the Int8 or the debug copy takes the staged path).
template <int COLS, bool ABSMAX, typename Release>
__device__ __forceinline__ void epilogue_warp_direct(const GemmArgs &a, uint32_t taddr, int64_t row0, int64_t col0,
                                                     const int32_t (&bqv)[COLS / 32], const float (&invv)[COLS / 32],
                                                     int32_t *bq_s, int lane, int nch, Release release, float &absmax_run)
{
    constexpr int NCHUNK = COLS / 32;
    const int g = lane >> 2, cq = 2 * (lane & 3);
    uint32_t v[32];  // v[16 h + 4 i + 2 r + c]: row 16 h + 8 r + g, column 8 i + cq + c of the block
#pragma unroll
    for (int ci = 0; ci < NCHUNK; ++ci) {
        if (ci >= nch) break;
        tmem_ld_16x256b_x4(taddr + (uint32_t)(32 * ci), v);
        tmem_ld_16x256b_x4(taddr + (16u << 16) + (uint32_t)(32 * ci), v + 16);
        tmem_ld_wait();
        if (ci + 1 == nch) release();
        const int64_t nb = col0 + 32 * ci;
        const float inv = invv[ci];
        if (nb >= a.N || row0 >= a.M) continue;  // warp-uniform: the block lies outside the matrix
        __syncwarp();
        bq_s[lane] = bqv[ci];
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int2 b = *reinterpret_cast<const int2 *>(bq_s + 8 * i + cq);
#pragma unroll
            for (int hr = 0; hr < 4; ++hr) {
                const int k = 16 * (hr >> 1) + 4 * i + 2 * (hr & 1);
                v[k] = (uint32_t)add_wrap((int32_t)v[k], b.x);
                v[k + 1] = (uint32_t)add_wrap((int32_t)v[k + 1], b.y);
            }
        }
        if (a.act == Q8_ACT_GELU) {
            const uint64_t inv2 = pack_f32x2(inv, inv);
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                const uint64_t y2 =
                    mul_f32x2(pack_f32x2(__int2float_rn((int32_t)v[j]), __int2float_rn((int32_t)v[j + 1])), inv2);
                float g0, g1;
                gelu_fast_x2(y2, g0, g1);
                v[j] = __float_as_uint(g0);
                v[j + 1] = __float_as_uint(g1);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__fmul_rn(__int2float_rn((int32_t)v[j]), inv));
        }
#pragma unroll
        for (int hr = 0; hr < 4; ++hr) {
            const int64_t row = row0 + 16 * (hr >> 1) + 8 * (hr & 1) + g;
            float *yrow = a.Y + row * a.N + nb + cq;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = 16 * (hr >> 1) + 4 * i + 2 * (hr & 1);
                if (row < a.M && nb + 8 * i + cq < a.N) {
                    const float y0 = __uint_as_float(v[k]), y1 = __uint_as_float(v[k + 1]);
                    if (ABSMAX) absmax_run = fmaxf(absmax_run, fmaxf(fabsf(y0), fabsf(y1)));
                    *reinterpret_cast<float2 *>(yrow + 8 * i) = make_float2(y0, y1);
                }
            }
        }
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn()
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

// A tensor map depends only on the base address, the extents and the box, and a serving loop calls with the same
// few buffers over and over, so the encoded maps are kept in a small per-thread table (direct-mapped on a hash of
// those fields): a hit saves the driver call, which matters for launch-bound small problems.
struct TmapKey {
    const void *base;
    int64_t d0, d1;
    int32_t box0, box1, kind;
    bool operator==(const TmapKey &o) const
    {
        return base == o.base && d0 == o.d0 && d1 == o.d1 && box0 == o.box0 && box1 == o.box1 && kind == o.kind;
    }
};
struct TmapSlot {
    TmapKey key;
    CUtensorMap map;
    bool valid = false;
};
constexpr int kTmapSlots = 64;

template <typename Encode>
inline bool cached_tmap(CUtensorMap *out, const TmapKey &key, Encode encode)
{
    static thread_local TmapSlot table[kTmapSlots];
    uint64_t h = reinterpret_cast<uintptr_t>(key.base) * 0x9E3779B97F4A7C15ull;
    h ^= (uint64_t)key.d0 * 0xC2B2AE3D27D4EB4Full + (uint64_t)key.d1 * 0x165667B19E3779F9ull +
         (uint64_t)(key.box1 * 131 + key.box0 * 7 + key.kind);
    TmapSlot &slot = table[(h >> 40) % kTmapSlots];
    if (slot.valid && slot.key == key) {
        *out = slot.map;
        return true;
    }
    if (!encode(out)) return false;
    slot.key = key;
    slot.map = *out;
    slot.valid = true;
    return true;
}

// Row-major int8 matrix [rows, K] as a 2-D tensor map with (128 x box_rows) boxes, 128-byte swizzle.
// Elements outside the matrix read as zero, which is what ragged M, N and K tails need.
inline bool make_tmap(CUtensorMap *map, const int8_t *base, int64_t rows, int64_t K, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    return cached_tmap(map, TmapKey{base, K, rows, BLOCK_K, box_rows, 0}, [&](CUtensorMap *m) {
        cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)K};
        cuuint32_t box[2] = {(cuuint32_t)BLOCK_K, (cuuint32_t)box_rows};
        cuuint32_t estr[2] = {1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Row-major fp32 output [M, N] as a tensor map of 32 x 32 boxes (128 bytes wide), 128-byte swizzle.
// Stores that reach past row M or column N are clipped by the hardware.
inline bool make_tmap_out(CUtensorMap *map, float *base, int64_t M, int64_t N)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    return cached_tmap(map, TmapKey{base, N, M, 32, 32, 1}, [&](CUtensorMap *m) {
        cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
        cuuint64_t strides[1] = {(cuuint64_t)N * 4};
        cuuint32_t box[2] = {32, 32};
        cuuint32_t estr[2] = {1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

// Row-major Int8 output [M, N] as a tensor map of (box_cols x 32) boxes: 64-byte rows with the 64-byte swizzle
// or 128-byte rows with the 128-byte swizzle.
inline bool make_tmap_out_q(CUtensorMap *map, int8_t *base, int64_t M, int64_t N, int box_cols)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    return cached_tmap(map, TmapKey{base, N, M, box_cols, 32, 2}, [&](CUtensorMap *m) {
        cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
        cuuint64_t strides[1] = {(cuuint64_t)N};
        cuuint32_t box[2] = {(cuuint32_t)box_cols, 32};
        cuuint32_t estr[2] = {1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  box_cols == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

inline int sm_count()
{
    static int n = [] {
        int dev = 0, v = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

}  // namespace gemm_detail
}  // namespace q8
