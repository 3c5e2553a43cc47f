// Generic Int8 GEMM + epilogue on CUDA cores (dp4a): any M, N, K and any alignment.
//
// q8_linear falls back to this kernel when the tensor-core kernel's TMA preconditions do not
// hold (K not a multiple of 16 bytes, operands not 16-byte aligned).  It computes exactly the
// same integers (Sec. 3: Int8 products accumulated in Int32 onto the Int32 bias) and applies the
// same epilogue arithmetic, so it also serves as an on-device cross-check of the fast kernel.

#include "q8_internal.cuh"

namespace q8 {

namespace {

constexpr int TM = 64, TN = 64, TK = 64;  // CTA tile; 256 threads, each owns a 4x4 block of outputs
constexpr int PAD = 4;                    // row pitch TK + 4 bytes keeps 4-byte alignment and skews banks

__global__ void __launch_bounds__(256) gemm_generic_kernel(GemmArgs a)
{
    __shared__ __align__(16) int8_t As[TM][TK + PAD];
    __shared__ __align__(16) int8_t Bs[TN][TK + PAD];

    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * TM, n0 = (int64_t)blockIdx.y * TN;
    int32_t acc[4][4] = {};

    for (int64_t k0 = 0; k0 < a.K; k0 += TK) {
        // stage the two tiles, zero-filled outside the matrices (zeros add nothing to the sum)
        for (int e = threadIdx.x; e < TM * TK; e += 256) {
            const int r = e / TK, c = e % TK;
            const int64_t gm = m0 + r, gn = n0 + r, gk = k0 + c;
            As[r][c] = (gm < a.M && gk < a.K) ? a.Xq[gm * a.K + gk] : (int8_t)0;
            Bs[r][c] = (gn < a.N && gk < a.K) ? a.Wq[gn * a.K + gk] : (int8_t)0;
        }
        __syncthreads();
#pragma unroll 4
        for (int k4 = 0; k4 < TK / 4; ++k4) {
            int32_t av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                av[i] = *reinterpret_cast<const int32_t *>(&As[ty * 4 + i][k4 * 4]);
                bv[i] = *reinterpret_cast<const int32_t *>(&Bs[tx * 4 + i][k4 * 4]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

    const float S_x = __ldg(a.S_x);
    const float S_y = a.Yq ? __ldg(a.S_y) : 1.0f;
    float am = 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int64_t n = n0 + tx * 4 + j;
        if (n >= a.N) continue;
        const float S_out = __fmul_rn(S_x, __ldg(a.S_w + (a.w_seg > 0 ? n / a.w_seg : 0)));
        const float inv = __fdiv_rn(1.0f, S_out);
        const int32_t bq = a.bias ? quantize_bias(__ldg(a.bias + n), S_out) : 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t m = m0 + ty * 4 + i;
            if (m >= a.M) continue;
            const int32_t v = add_wrap(acc[i][j], bq);
            if (a.dbg_acc) a.dbg_acc[m * a.N + n] = v;
            const float y = finish_output(v, inv, a.act);
            am = fmaxf(am, fabsf(y));
            if (a.Y) a.Y[m * a.N + n] = y;
            if (a.Yq) a.Yq[m * a.N + n] = (int8_t)quantize_value(y, S_y);
        }
    }
    if (a.y_absmax) warp_fold_absmax(am, a.y_absmax);
}

}  // namespace

cudaError_t launch_gemm_generic(const GemmArgs &a, cudaStream_t s)
{
    dim3 grid((unsigned)((a.M + TM - 1) / TM), (unsigned)((a.N + TN - 1) / TN));
    if (grid.y > 65535u) return cudaErrorInvalidConfiguration;
    gemm_generic_kernel<<<grid, 256, 0, s>>>(a);
    LaunchInfo &li = last_launch_info();
    li.gemm_kernel = 2;
    li.block_n = TN;
    li.grid = (int)(grid.x * grid.y);
    li.launches += 1;
    return cudaGetLastError();
}

}  // namespace q8
