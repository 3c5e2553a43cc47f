// FP32 operations of the BERT encoder that Q8BERT leaves unquantised (Sec. 3: Softmax, Layer
// Normalization and GELU stay in FP32; the attention score / context products are not FC layers):
// residual add + LayerNorm, and scaled-dot-product self-attention.  They exist so that a whole
// encoder forward can run through this library; the quantised path proper is in the other files.

#include <math.h>

#include "q8_internal.cuh"

namespace q8 {

namespace {

// ------------------------------------------------------------------ out = LayerNorm(x + r1 + r2) * gamma + beta
// One CTA per row.  The summed row is kept in shared memory, so the inputs are read once; mean and
// variance are the two-pass forms (sum, then sum of squared deviations), reduced through warp shuffles.
constexpr int kLnThreads = 256;
constexpr int kLnCtasPerSm = 4;  // CTAs per SM of the warp-per-row kernel (64 registers x 256 threads each)

__device__ __forceinline__ float block_sum(float v, float *scratch)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();  // scratch may still be read from the previous reduction
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.0f;
#pragma unroll
    for (int w = 0; w < kLnThreads / 32; ++w) t += scratch[w];
    return t;
}

__global__ void __launch_bounds__(kLnThreads) add_layernorm_kernel(const float *__restrict__ x,
                                                                   const float *__restrict__ r1,
                                                                   const float *__restrict__ r2,
                                                                   const float *__restrict__ gamma,
                                                                   const float *__restrict__ beta, float eps, int64_t H,
                                                                   float *__restrict__ out, const float *__restrict__ S_q,
                                                                   int8_t *__restrict__ out_q, uint32_t *__restrict__ amax)
{
    extern __shared__ float row[];
    __shared__ float scratch[kLnThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * H;
    float s = 0.0f;
    for (int64_t h = threadIdx.x; h < H; h += kLnThreads) {
        float v = x[base + h];
        if (r1) v += r1[base + h];
        if (r2) v += r2[base + h];
        row[h] = v;
        s += v;
    }
    const float mean = block_sum(s, scratch) / (float)H;
    float q = 0.0f;
    for (int64_t h = threadIdx.x; h < H; h += kLnThreads) {
        const float d = row[h] - mean;
        q += d * d;
    }
    const float var = block_sum(q, scratch) / (float)H;
    const float rstd = 1.0f / sqrtf(var + eps);
    const float Sq = out_q ? __ldg(S_q) : 1.0f;
    float am = 0.0f;
    for (int64_t h = threadIdx.x; h < H; h += kLnThreads) {
        const float g = gamma ? gamma[h] : 1.0f, b = beta ? beta[h] : 0.0f;
        const float y = (row[h] - mean) * rstd * g + b;
        am = fmaxf(am, fabsf(y));
        if (out) out[base + h] = y;
        // the same fp32 value, quantised for the next quantised layer (Eq. 1 at that layer's scale)
        if (out_q) out_q[base + h] = (int8_t)quantize_value(y, Sq);
    }
    if (amax) warp_fold_absmax(am, amax);  // max|y| for a dynamically quantised consumer (Sec. 4.1)
}

// Vector form for H % 4 == 0, H <= 4096 and 16-byte aligned rows: the row lives in registers (up to four
// float4 per thread), every access is a 16-byte one, and the Int8 copy is written four values at a time.
__global__ void __launch_bounds__(kLnThreads) add_layernorm_vec_kernel(const float *__restrict__ x,
                                                                       const float *__restrict__ r1,
                                                                       const float *__restrict__ r2,
                                                                       const float *__restrict__ gamma,
                                                                       const float *__restrict__ beta, float eps,
                                                                       int64_t H, float *__restrict__ out,
                                                                       const float *__restrict__ S_q,
                                                                       int8_t *__restrict__ out_q, uint32_t *__restrict__ amax)
{
    __shared__ float scratch[kLnThreads / 32];
    const int64_t base4 = (int64_t)blockIdx.x * (H >> 2);
    const int n4 = (int)(H >> 2);
    const float4 *x4 = reinterpret_cast<const float4 *>(x) + base4;
    const float4 *a4 = r1 ? reinterpret_cast<const float4 *>(r1) + base4 : nullptr;
    const float4 *b4 = r2 ? reinterpret_cast<const float4 *>(r2) + base4 : nullptr;
    float4 v[4];
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = threadIdx.x + kLnThreads * i;
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < n4) {
            v[i] = x4[c];
            if (a4) { const float4 t = a4[c]; v[i].x += t.x; v[i].y += t.y; v[i].z += t.z; v[i].w += t.w; }
            if (b4) { const float4 t = b4[c]; v[i].x += t.x; v[i].y += t.y; v[i].z += t.z; v[i].w += t.w; }
            s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
        }
    }
    const float mean = block_sum(s, scratch) / (float)H;
    float q = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (threadIdx.x + kLnThreads * i < n4) {
            const float dx = v[i].x - mean, dy = v[i].y - mean, dz = v[i].z - mean, dw = v[i].w - mean;
            q += (dx * dx + dy * dy) + (dz * dz + dw * dw);
        }
    const float var = block_sum(q, scratch) / (float)H;
    const float rstd = 1.0f / sqrtf(var + eps);
    const float Sq = out_q ? __ldg(S_q) : 1.0f;
    float am = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = threadIdx.x + kLnThreads * i;
        if (c >= n4) continue;
        const float4 g = gamma ? reinterpret_cast<const float4 *>(gamma)[c] : make_float4(1.f, 1.f, 1.f, 1.f);
        const float4 b = beta ? reinterpret_cast<const float4 *>(beta)[c] : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 y;
        y.x = (v[i].x - mean) * rstd * g.x + b.x;
        y.y = (v[i].y - mean) * rstd * g.y + b.y;
        y.z = (v[i].z - mean) * rstd * g.z + b.z;
        y.w = (v[i].w - mean) * rstd * g.w + b.w;
        am = fmaxf(fmaxf(am, fmaxf(fabsf(y.x), fabsf(y.y))), fmaxf(fabsf(y.z), fabsf(y.w)));
        if (out) reinterpret_cast<float4 *>(out)[base4 + c] = y;
        if (out_q) reinterpret_cast<uint32_t *>(out_q)[base4 + c] = quantize_pack4(y.x, y.y, y.z, y.w, Sq);
    }
    if (amax) warp_fold_absmax(am, amax);
}

// One warp per row for H <= 1024 (BERT's hidden sizes): up to eight float4 per lane, both moments reduced with
// shuffles only, eight rows per CTA, so there is no block-level barrier at all.
__global__ void __launch_bounds__(kLnThreads, kLnCtasPerSm) add_layernorm_warp_kernel(const float *__restrict__ x,
                                                                        const float *__restrict__ r1,
                                                                        const float *__restrict__ r2,
                                                                        const float *__restrict__ gamma,
                                                                        const float *__restrict__ beta, float eps,
                                                                        int64_t rows, int64_t H, float *__restrict__ out,
                                                                        const float *__restrict__ S_q,
                                                                        int8_t *__restrict__ out_q, uint32_t *__restrict__ amax)
{
    grid_dependency_release_next(rows * H <= kSmallProblemElems);
    grid_dependency_wait();  // launched so that its start may overlap the tail of the kernel before it
    const int lane = threadIdx.x & 31;
    const int n4 = (int)(H >> 2);
    const float Sq = out_q ? __ldg(S_q) : 1.0f;
    float am = 0.0f;  // running max|y| of this lane over all rows of the warp
    // the grid is sized to the device and every warp walks rows with a grid stride (no partial last wave)
    for (int64_t row = (int64_t)blockIdx.x * (kLnThreads / 32) + (threadIdx.x >> 5); row < rows;
         row += (int64_t)gridDim.x * (kLnThreads / 32)) {
    const int64_t base4 = row * n4;
    const float4 *x4 = reinterpret_cast<const float4 *>(x) + base4;
    const float4 *a4 = r1 ? reinterpret_cast<const float4 *>(r1) + base4 : nullptr;
    const float4 *b4 = r2 ? reinterpret_cast<const float4 *>(r2) + base4 : nullptr;
    float4 v[8];
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int c = lane + 32 * i;
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < n4) {
            v[i] = __ldg(x4 + c);
            if (a4) { const float4 t = __ldg(a4 + c); v[i].x += t.x; v[i].y += t.y; v[i].z += t.z; v[i].w += t.w; }
            if (b4) { const float4 t = __ldg(b4 + c); v[i].x += t.x; v[i].y += t.y; v[i].z += t.z; v[i].w += t.w; }
            s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mean = s / (float)H;
    float q = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (lane + 32 * i < n4) {
            const float dx = v[i].x - mean, dy = v[i].y - mean, dz = v[i].z - mean, dw = v[i].w - mean;
            q += (dx * dx + dy * dy) + (dz * dz + dw * dw);
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    const float rstd = 1.0f / sqrtf(q / (float)H + eps);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int c = lane + 32 * i;
        if (c >= n4) continue;
        const float4 g = gamma ? __ldg(reinterpret_cast<const float4 *>(gamma) + c) : make_float4(1.f, 1.f, 1.f, 1.f);
        const float4 b = beta ? __ldg(reinterpret_cast<const float4 *>(beta) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 y;
        y.x = (v[i].x - mean) * rstd * g.x + b.x;
        y.y = (v[i].y - mean) * rstd * g.y + b.y;
        y.z = (v[i].z - mean) * rstd * g.z + b.z;
        y.w = (v[i].w - mean) * rstd * g.w + b.w;
        am = fmaxf(fmaxf(am, fmaxf(fabsf(y.x), fabsf(y.y))), fmaxf(fabsf(y.z), fabsf(y.w)));
        if (out) reinterpret_cast<float4 *>(out)[base4 + c] = y;
        if (out_q) reinterpret_cast<uint32_t *>(out_q)[base4 + c] = quantize_pack4(y.x, y.y, y.z, y.w, Sq);
    }
    }
    if (amax) warp_fold_absmax(am, amax);  // one atomic per warp: max|y| for a dynamically quantised consumer (Sec. 4.1)
}

// ------------------------------------------------------------------ self-attention, head dimension 64, no mask
// ctx[b, i, head] = softmax_j(q_i . k_j / 8) v_j with q, k, v read from the fused projection
// qkv[T, 3H] = [q | k | v].  One CTA per (64 queries, head, sequence); keys and values stream through
// shared memory in tiles of 64 with the running-max / running-sum form of softmax, all in fp32.
// Thread (ty, tx) of the 16 x 16 CTA owns rows {2ty, 2ty+1, 2ty+32, 2ty+33} x columns {2tx, 2tx+1, 2tx+32,
// 2tx+33} of the 64 x 64 score tile and of the output tile, so its operands are two 8-byte loads each and
// consecutive lanes touch consecutive banks.  Q, K and P are held transposed with a pitch of 66 floats.
constexpr int kD = 64, kTile = 64, kPitch = 66;
constexpr int kAttnSmemBytes = (3 * kD * kPitch + kTile * kD) * (int)sizeof(float);

__device__ __forceinline__ int own_index(int t, int a) { return 2 * t + (a & 1) + 32 * (a >> 1); }

__global__ void __launch_bounds__(256) attention_kernel(const float *__restrict__ qkv, int64_t S, int64_t H,
                                                        float scale, float *__restrict__ ctx,
                                                        const float *__restrict__ S_q, int8_t *__restrict__ ctx_q,
                                                        uint32_t *__restrict__ amax)
{
    extern __shared__ __align__(16) float attn_smem[];
    float(*Qt)[kPitch] = reinterpret_cast<float(*)[kPitch]>(attn_smem);                    // Qt[d][i]
    float(*Kt)[kPitch] = reinterpret_cast<float(*)[kPitch]>(attn_smem + kD * kPitch);       // Kt[d][j]
    float(*Pt)[kPitch] = reinterpret_cast<float(*)[kPitch]>(attn_smem + 2 * kD * kPitch);   // Pt[j][i]
    float(*Vs)[kD] = reinterpret_cast<float(*)[kD]>(attn_smem + 3 * kD * kPitch);           // Vs[j][d]

    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t q0 = (int64_t)blockIdx.x * kTile, head = blockIdx.y, seq = blockIdx.z;
    const int64_t row_pitch = 3 * H;
    const float *base = qkv + seq * S * row_pitch + head * kD;

    // queries of this CTA, pre-scaled by log2(e) / sqrt(d) so that the softmax can use exp2 directly, transposed;
    // rows past the sequence end are zero
    for (int e = threadIdx.x; e < kTile * kD; e += 256) {
        const int i = e / kD, d = e % kD;
        Qt[d][i] = (q0 + i < S) ? base[(q0 + i) * row_pitch + d] * scale : 0.0f;
    }

    float o[4][4] = {};
    float m[4], l[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        m[a] = -INFINITY;
        l[a] = 0.0f;
    }

    // The next key / value tile is fetched into registers while the current one is being used, so the global
    // load latency overlaps the arithmetic.  Element e = tid + 256 i of a tile is (key j = e / 64, feature d = e % 64).
    float kreg[16], vreg[16];
    auto fetch_tile = [&](int64_t j0) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int e = threadIdx.x + 256 * i;
            const int j = e / kD, d = e % kD;
            const bool ok = j0 + j < S;
            kreg[i] = ok ? __ldg(base + (j0 + j) * row_pitch + H + d) : 0.0f;
            vreg[i] = ok ? __ldg(base + (j0 + j) * row_pitch + 2 * H + d) : 0.0f;
        }
    };
    fetch_tile(0);

    for (int64_t j0 = 0; j0 < S; j0 += kTile) {
        __syncthreads();  // previous tile fully consumed (and Qt written, on the first pass)
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int e = threadIdx.x + 256 * i;
            Kt[e % kD][e / kD] = kreg[i];
            Vs[e / kD][e % kD] = vreg[i];
        }
        __syncthreads();
        if (j0 + kTile < S) fetch_tile(j0 + kTile);

        float s[4][4] = {};
#pragma unroll 8
        for (int d = 0; d < kD; ++d) {
            const float2 q01 = *reinterpret_cast<const float2 *>(&Qt[d][2 * ty]);
            const float2 q23 = *reinterpret_cast<const float2 *>(&Qt[d][2 * ty + 32]);
            const float2 k01 = *reinterpret_cast<const float2 *>(&Kt[d][2 * tx]);
            const float2 k23 = *reinterpret_cast<const float2 *>(&Kt[d][2 * tx + 32]);
            const float qv[4] = {q01.x, q01.y, q23.x, q23.y}, kv[4] = {k01.x, k01.y, k23.x, k23.y};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) s[a][b] = fmaf(qv[a], kv[b], s[a][b]);
        }
        // keys past the sequence end do not take part
#pragma unroll
        for (int b = 0; b < 4; ++b)
            if (j0 + own_index(tx, b) >= S) {
#pragma unroll
                for (int a = 0; a < 4; ++a) s[a][b] = -INFINITY;
            }
        // running max / sum per query row (a row's 64 scores live in the 16 threads that share ty)
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float mx = fmaxf(fmaxf(s[a][0], s[a][1]), fmaxf(s[a][2], s[a][3]));
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            const float m_new = fmaxf(m[a], mx);
            const float corr = exp2f(m[a] - m_new);  // 2^(-inf) = 0 on the first tile
            float sum = 0.0f;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                s[a][b] = exp2f(s[a][b] - m_new);
                sum += s[a][b];
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            l[a] = l[a] * corr + sum;
            m[a] = m_new;
#pragma unroll
            for (int b = 0; b < 4; ++b) o[a][b] *= corr;
        }
        // probabilities to shared memory (transposed), then O += P V
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int j = own_index(tx, b);
            *reinterpret_cast<float2 *>(&Pt[j][2 * ty]) = make_float2(s[0][b], s[1][b]);
            *reinterpret_cast<float2 *>(&Pt[j][2 * ty + 32]) = make_float2(s[2][b], s[3][b]);
        }
        __syncthreads();
#pragma unroll 8
        for (int j = 0; j < kTile; ++j) {
            const float2 p01 = *reinterpret_cast<const float2 *>(&Pt[j][2 * ty]);
            const float2 p23 = *reinterpret_cast<const float2 *>(&Pt[j][2 * ty + 32]);
            const float2 v01 = *reinterpret_cast<const float2 *>(&Vs[j][2 * tx]);
            const float2 v23 = *reinterpret_cast<const float2 *>(&Vs[j][2 * tx + 32]);
            const float pv[4] = {p01.x, p01.y, p23.x, p23.y}, vv[4] = {v01.x, v01.y, v23.x, v23.y};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) o[a][b] = fmaf(pv[a], vv[b], o[a][b]);
        }
    }

    const int64_t obase = seq * S * H + head * kD;
    const float Sq = ctx_q ? __ldg(S_q) : 1.0f;
    float am = 0.0f;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int64_t i = q0 + own_index(ty, a);
        if (i >= S) continue;
        const float inv = 1.0f / l[a];
        const float y0 = o[a][0] * inv, y1 = o[a][1] * inv, y2 = o[a][2] * inv, y3 = o[a][3] * inv;
        am = fmaxf(fmaxf(am, fmaxf(fabsf(y0), fabsf(y1))), fmaxf(fabsf(y2), fabsf(y3)));
        const int64_t at = obase + i * H + 2 * tx;
        if (ctx) {
            *reinterpret_cast<float2 *>(ctx + at) = make_float2(y0, y1);
            *reinterpret_cast<float2 *>(ctx + at + 32) = make_float2(y2, y3);
        }
        if (ctx_q) {  // the same fp32 values, quantised for the next quantised layer
            ctx_q[at] = (int8_t)quantize_value(y0, Sq);
            ctx_q[at + 1] = (int8_t)quantize_value(y1, Sq);
            ctx_q[at + 32] = (int8_t)quantize_value(y2, Sq);
            ctx_q[at + 33] = (int8_t)quantize_value(y3, Sq);
        }
    }
    if (amax) warp_fold_absmax(am, amax);
}

}  // namespace

cudaError_t launch_add_layernorm(const float *x, const float *r1, const float *r2, const float *gamma,
                                 const float *beta, float eps, int64_t rows, int64_t H, float *out, const float *S_q,
                                 int8_t *out_q, uint32_t *amax, cudaStream_t s)
{
    if (rows <= 0 || H <= 0) return cudaSuccess;
    auto al16 = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    const bool vec = (H % 4 == 0) && H <= 4 * 4 * kLnThreads && al16(x) && al16(r1) && al16(r2) && al16(gamma) &&
                     al16(beta) && al16(out) && (reinterpret_cast<uintptr_t>(out_q) & 3u) == 0;
    if (vec && H <= 1024) {
        const int64_t want = (rows + kLnThreads / 32 - 1) / (kLnThreads / 32);
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int64_t cap = (int64_t)(sms > 0 ? sms : 148) * kLnCtasPerSm;
        const unsigned blocks = (unsigned)(want < cap ? want : cap);
        return launch_overlapping_tail(add_layernorm_warp_kernel, dim3(blocks), dim3(kLnThreads), 0, s, x, r1, r2, gamma, beta,
                                       eps, rows, H, out, S_q, out_q, amax);
    } else if (vec) {
        add_layernorm_vec_kernel<<<(unsigned)rows, kLnThreads, 0, s>>>(x, r1, r2, gamma, beta, eps, H, out, S_q, out_q, amax);
    } else {
        add_layernorm_kernel<<<(unsigned)rows, kLnThreads, (size_t)H * sizeof(float), s>>>(x, r1, r2, gamma, beta, eps,
                                                                                           H, out, S_q, out_q, amax);
    }
    return cudaGetLastError();
}

cudaError_t launch_attention(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                             int8_t *ctx_q, uint32_t *amax, cudaStream_t s)
{
    if (B <= 0 || S <= 0 || heads <= 0) return cudaSuccess;
    if (attention_tc_supported(qkv, S, heads, ctx, ctx_q))
        return launch_attention_tc(qkv, B, S, heads, ctx, S_q, ctx_q, amax, s);
    static bool attr_set[64] = {};  // opt-in shared-memory size: per device, per function
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    dim3 grid((unsigned)((S + kTile - 1) / kTile), (unsigned)heads, (unsigned)B);
    attention_kernel<<<grid, 256, kAttnSmemBytes, s>>>(qkv, S, heads * kD, 1.4426950408889634f / 8.0f, ctx, S_q, ctx_q, amax);
    return cudaGetLastError();
}

}  // namespace q8
