// extern "C" entry points of libq8: argument validation, kernel selection and launches.
// Nothing here computes; every step of the path runs in the kernels of the other files.

#include <limits.h>

#include "q8_internal.cuh"

namespace q8 {

LaunchInfo &last_launch_info()
{
    static thread_local LaunchInfo info;
    return info;
}

namespace {

inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

#define Q8_CUDA_TRY(expr)                      \
    do {                                       \
        cudaError_t e__ = (expr);              \
        if (e__ != cudaSuccess) return Q8_ERR_CUDA; \
    } while (0)

// Eq. 1 with either a given scale or the dynamic one of Eq. 3 / Sec. 4.1 (scratch == output scale word).
q8_status quantize_tensor(const float *X, int64_t numel, const float *S_given, int8_t *Xq, int8_t *Xq_copy,
                          float *S_dyn, bool S_dyn_is_zero, int32_t *status, cudaStream_t s)
{
    LaunchInfo &li = last_launch_info();
    const float *S = S_given;
    if (S_given == nullptr) {
        // The scale word first holds the float bits of the running maximum, then the scale itself.
        if (!S_dyn_is_zero) Q8_CUDA_TRY(cudaMemsetAsync(S_dyn, 0, sizeof(float), s));
        Q8_CUDA_TRY(launch_absmax(X, numel, reinterpret_cast<uint32_t *>(S_dyn), s));
        Q8_CUDA_TRY(launch_scale_from_absmax(reinterpret_cast<const uint32_t *>(S_dyn), S_dyn, status, s));
        li.launches += numel > 0 ? 2 : 1;
        S = S_dyn;
    }
    Q8_CUDA_TRY(launch_quantize(X, numel, S, Xq, Xq_copy, s, nullptr, S_given != nullptr ? status : nullptr));
    li.launches += numel > 0 ? 1 : 0;
    return Q8_OK;
}

q8_status check_gemm_shape(int64_t M, int64_t N, int64_t K)
{
    if (M < 0 || N < 0 || K < 0) return Q8_ERR_SHAPE;
    if (M == 0 || N == 0) return Q8_OK;
    if (K == 0) return Q8_ERR_SHAPE;
    if (K > Q8_MAX_K) return Q8_ERR_OVERFLOW;
    if (M > (int64_t)INT_MAX || N > (int64_t)INT_MAX) return Q8_ERR_SHAPE;
    return Q8_OK;
}

q8_status run_gemm(const GemmArgs &g, bool force_generic, cudaStream_t s)
{
    if (!force_generic && tcgen05_gemm_supported(g)) {
        Q8_CUDA_TRY(launch_gemm_tcgen05(g, s));
    } else {
        Q8_CUDA_TRY(launch_gemm_generic(g, s));
    }
    return Q8_OK;
}

}  // namespace

q8_status linear_impl(const float *X, const int8_t *Wq, const float *S_w, const float *S_x, const float *bias, int act,
                      float *Y, int64_t M, int64_t N, int64_t K, void *workspace, size_t workspace_bytes,
                      int8_t *dbg_Xq, int32_t *dbg_acc, void *stream, bool force_generic, int8_t *Yq,
                      const float *S_y, int64_t w_seg, const uint32_t *x_absmax, uint32_t *y_absmax)
{
    last_launch_info() = LaunchInfo();
    q8_status st = check_gemm_shape(M, N, K);
    if (st != Q8_OK) return st;
    if (M == 0 || N == 0) return Q8_OK;  // nothing to compute; empty tensors may carry NULL pointers
    if (!X || !Wq || !S_w || !workspace) return Q8_ERR_NULL;
    if (!Y && !Yq) return Q8_ERR_NULL;
    if (Yq && !S_y) return Q8_ERR_NULL;
    if (S_y && !aligned_to(S_y, 4)) return Q8_ERR_ALIGN;
    if (w_seg < 0) return Q8_ERR_SHAPE;
    if (act != Q8_ACT_NONE && act != Q8_ACT_GELU) return Q8_ERR_ARG;
    if (!aligned_to(X, 4) || !aligned_to(Y, 4) || !aligned_to(S_w, 4) || (S_x && !aligned_to(S_x, 4)) ||
        (bias && !aligned_to(bias, 4)) || (dbg_acc && !aligned_to(dbg_acc, 4)) || !aligned_to(workspace, 256))
        return Q8_ERR_ALIGN;
    if (workspace_bytes < q8_linear_workspace_bytes(M, N, K)) return Q8_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WorkspaceHeader *hdr = static_cast<WorkspaceHeader *>(workspace);
    int8_t *Xq = static_cast<int8_t *>(workspace) + kWorkspaceHeaderBytes;
    // Eq. 1.  With a given scale the quantise kernel itself starts the call's status word at zero (no separate
    // clearing operation in the stream); with the Sec. 4.1 dynamic scale (S_x NULL) the header is zeroed first, then
    // come the abs-max pass and one kernel that turns the maximum into the scale and quantises with it.
    if ((x_absmax && !aligned_to(x_absmax, 4)) || (y_absmax && !aligned_to(y_absmax, 4))) return Q8_ERR_ALIGN;
    if (S_x != nullptr) {
        Q8_CUDA_TRY(launch_quantize(X, M * K, S_x, Xq, dbg_Xq, s, &hdr->status));
        last_launch_info().launches += 1;
    } else if (x_absmax != nullptr) {
        // Sec. 4.1 with max|X| already known (folded into a device word by the kernel that produced X): one kernel
        // derives the scale from it, publishes it in the header and quantises; it also starts the status word at zero.
        Q8_CUDA_TRY(launch_quantize_dynamic(X, M * K, x_absmax, &hdr->S_x_dyn, &hdr->status, Xq, dbg_Xq, s, true));
        last_launch_info().launches += 1;
    } else if (quantize_dynamic_small_supported(X, M * K, Xq, dbg_Xq)) {
        // a small activation (up to 256 x 768): abs-max, scale and Eq. 1 in one launch of one cluster, no memset
        Q8_CUDA_TRY(launch_quantize_dynamic_small(X, M * K, &hdr->S_x_dyn, &hdr->status, Xq, dbg_Xq, s));
        last_launch_info().launches += 1;
    } else {
        Q8_CUDA_TRY(cudaMemsetAsync(hdr, 0, sizeof(WorkspaceHeader), s));
        Q8_CUDA_TRY(launch_absmax(X, M * K, &hdr->absmax_bits, s));
        Q8_CUDA_TRY(launch_quantize_dynamic(X, M * K, &hdr->absmax_bits, &hdr->S_x_dyn, &hdr->status, Xq, dbg_Xq, s));
        last_launch_info().launches += 2;
    }

    GemmArgs g;
    g.Xq = Xq;
    g.Wq = Wq;
    g.S_x = S_x ? S_x : &hdr->S_x_dyn;
    g.S_w = S_w;
    g.w_seg = w_seg;
    g.bias = bias;
    g.Y = Y;
    g.Yq = Yq;
    g.S_y = S_y;
    g.dbg_acc = dbg_acc;
    g.y_absmax = y_absmax;
    g.status = &hdr->status;
    g.M = M;
    g.N = N;
    g.K = K;
    g.act = act;
    return run_gemm(g, force_generic, s);
}


}  // namespace q8

using namespace q8;

extern "C" {

q8_status q8_quantize_weight(const float *W, int64_t N, int64_t K, int8_t *Wq, float *S_w, int32_t *dev_status,
                             void *stream)
{
    last_launch_info() = LaunchInfo();
    if (!S_w) return Q8_ERR_NULL;
    if (N < 0 || K < 0) return Q8_ERR_SHAPE;
    if (N > 0 && K > 0 && (!W || !Wq)) return Q8_ERR_NULL;
    if (N > 0 && K > 0 && N > (int64_t)LLONG_MAX / K) return Q8_ERR_SHAPE;
    if (!aligned_to(W, 4) || !aligned_to(S_w, 4) || (dev_status && !aligned_to(dev_status, 4))) return Q8_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (N == 0 || K == 0) {
        const float one = 1.0f;
        Q8_CUDA_TRY(cudaMemcpyAsync(S_w, &one, sizeof(float), cudaMemcpyHostToDevice, s));
        Q8_CUDA_TRY(cudaStreamSynchronize(s));  // `one` lives on this stack frame
        return Q8_OK;
    }
    return quantize_tensor(W, N * K, nullptr, Wq, nullptr, S_w, false, dev_status, s);
}

q8_status q8_quantize_activation(const float *X, int64_t numel, const float *S_x, int8_t *Xq, float *S_x_used,
                                 int32_t *dev_status, void *stream)
{
    last_launch_info() = LaunchInfo();
    if (numel < 0) return Q8_ERR_SHAPE;
    if (numel > 0 && (!X || !Xq)) return Q8_ERR_NULL;
    if (!S_x && !S_x_used) return Q8_ERR_NULL;
    if (!aligned_to(X, 4) || (S_x && !aligned_to(S_x, 4)) || (S_x_used && !aligned_to(S_x_used, 4)) ||
        (dev_status && !aligned_to(dev_status, 4)))
        return Q8_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    q8_status st = quantize_tensor(X, numel, S_x, Xq, nullptr, S_x_used, false, dev_status, s);
    if (st != Q8_OK) return st;
    if (S_x && S_x_used && S_x_used != S_x)
        Q8_CUDA_TRY(cudaMemcpyAsync(S_x_used, S_x, sizeof(float), cudaMemcpyDeviceToDevice, s));
    return Q8_OK;
}

q8_status q8_fake_quantize(const float *X, int64_t numel, const float *S, float *Xhat, void *stream)
{
    last_launch_info() = LaunchInfo();
    if (numel < 0) return Q8_ERR_SHAPE;
    if (numel == 0) return Q8_OK;
    if (!X || !S || !Xhat) return Q8_ERR_NULL;
    if (!aligned_to(X, 4) || !aligned_to(S, 4) || !aligned_to(Xhat, 4)) return Q8_ERR_ALIGN;
    Q8_CUDA_TRY(launch_fake_quantize(X, numel, S, Xhat, static_cast<cudaStream_t>(stream)));
    last_launch_info().launches = 1;
    return Q8_OK;
}

q8_status q8_ste_backward(const float *grad_out, int64_t numel, float *grad_in, void *stream)
{
    last_launch_info() = LaunchInfo();
    if (numel < 0) return Q8_ERR_SHAPE;
    if (numel == 0 || grad_in == grad_out) return Q8_OK;  // the estimator is the identity: in place is a no-op
    if (!grad_out || !grad_in) return Q8_ERR_NULL;
    Q8_CUDA_TRY(cudaMemcpyAsync(grad_in, grad_out, (size_t)numel * sizeof(float), cudaMemcpyDeviceToDevice,
                                static_cast<cudaStream_t>(stream)));
    return Q8_OK;
}

size_t q8_calibrate_state_bytes(void) { return sizeof(CalibState); }

q8_status q8_calibrate(const float *X, int64_t numel, float decay, void *state, void *stream)
{
    last_launch_info() = LaunchInfo();
    if (!state) return Q8_ERR_NULL;
    if (numel < 0) return Q8_ERR_SHAPE;
    if (numel > 0 && !X) return Q8_ERR_NULL;
    if (!(decay >= 0.0f && decay < 1.0f)) return Q8_ERR_ARG;
    if (!aligned_to(X, 4) || !aligned_to(state, 16)) return Q8_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CalibState *st = static_cast<CalibState *>(state);
    if (numel == 0) return Q8_OK;  // an empty batch is no observation of max|x|: the running state stays as it is
    Q8_CUDA_TRY(launch_absmax(X, numel, &st->scratch_bits, s));
    Q8_CUDA_TRY(launch_ema_update(st, decay, s));
    last_launch_info().launches = 2;
    return Q8_OK;
}

size_t q8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K)
{
    (void)N;
    if (M < 0 || K < 0) return 0;
    return kWorkspaceHeaderBytes + round_up((size_t)M * (size_t)K, 256);
}

q8_status q8_linear(const float *X, const int8_t *Wq, const float *S_w, const float *S_x, const float *bias, int act,
                    float *Y, int64_t M, int64_t N, int64_t K, void *workspace, size_t workspace_bytes,
                    int8_t *dbg_Xq, int32_t *dbg_acc, void *stream)
{
    return linear_impl(X, Wq, S_w, S_x, bias, act, Y, M, N, K, workspace, workspace_bytes, dbg_Xq, dbg_acc, stream,
                       false);
}

q8_status q8_linear_generic(const float *X, const int8_t *Wq, const float *S_w, const float *S_x, const float *bias,
                            int act, float *Y, int64_t M, int64_t N, int64_t K, void *workspace,
                            size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc, void *stream)
{
    return linear_impl(X, Wq, S_w, S_x, bias, act, Y, M, N, K, workspace, workspace_bytes, dbg_Xq, dbg_acc, stream,
                       true);
}

// Body of q8_linear_q / q8_linear_q_requant.
static q8_status linear_q_impl(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w,
                               const float *bias, int act, float *Y, int8_t *Yq, const float *S_y, int64_t M, int64_t N,
                               int64_t K, int32_t *dbg_acc, int32_t *dev_status, void *stream, int64_t w_seg = 0)
{
    last_launch_info() = LaunchInfo();
    q8_status st = check_gemm_shape(M, N, K);
    if (st != Q8_OK) return st;
    if (M == 0 || N == 0) return Q8_OK;
    if (!Xq || !S_x || !Wq || !S_w || (!Y && !Yq) || (Yq && !S_y)) return Q8_ERR_NULL;
    if (S_y && !aligned_to(S_y, 4)) return Q8_ERR_ALIGN;
    if (act != Q8_ACT_NONE && act != Q8_ACT_GELU) return Q8_ERR_ARG;
    if (!aligned_to(Y, 4) || !aligned_to(S_w, 4) || !aligned_to(S_x, 4) || (bias && !aligned_to(bias, 4)) ||
        (dbg_acc && !aligned_to(dbg_acc, 4)) || (dev_status && !aligned_to(dev_status, 4)))
        return Q8_ERR_ALIGN;
    GemmArgs g;
    g.Xq = Xq;
    g.Wq = Wq;
    g.S_x = S_x;
    g.S_w = S_w;
    g.w_seg = w_seg < 0 ? 0 : w_seg;
    g.bias = bias;
    g.Y = Y;
    g.Yq = Yq;
    g.S_y = S_y;
    g.dbg_acc = dbg_acc;
    g.status = dev_status;
    g.M = M;
    g.N = N;
    g.K = K;
    g.act = act;
    return run_gemm(g, false, static_cast<cudaStream_t>(stream));
}

q8_status q8_linear_q(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w, const float *bias,
                      int act, float *Y, int64_t M, int64_t N, int64_t K, int32_t *dbg_acc, int32_t *dev_status,
                      void *stream)
{
    if (M > 0 && N > 0 && !Y) return Q8_ERR_NULL;
    return linear_q_impl(Xq, S_x, Wq, S_w, bias, act, Y, nullptr, nullptr, M, N, K, dbg_acc, dev_status, stream);
}

q8_status q8_linear_q_requant(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w,
                              const float *bias, int act, const float *S_y, int8_t *Yq, float *Y, int64_t M, int64_t N,
                              int64_t K, int32_t *dbg_acc, int32_t *dev_status, void *stream)
{
    if (M > 0 && N > 0 && !Yq) return Q8_ERR_NULL;
    return linear_q_impl(Xq, S_x, Wq, S_w, bias, act, Y, Yq, S_y, M, N, K, dbg_acc, dev_status, stream);
}

q8_status q8_quantize_weight_segments(const float *W, int64_t N, int64_t K, int64_t seg_rows, int8_t *Wq, float *S_w,
                                      int32_t *dev_status, void *stream)
{
    if (seg_rows <= 0 || N < 0 || K < 0) return Q8_ERR_SHAPE;
    int launches = 0;
    for (int64_t r0 = 0, seg = 0; r0 < N; r0 += seg_rows, ++seg) {
        const int64_t rows = (N - r0 < seg_rows) ? N - r0 : seg_rows;
        q8_status st = q8_quantize_weight(W ? W + r0 * K : nullptr, rows, K, Wq ? Wq + r0 * K : nullptr,
                                          S_w ? S_w + seg : nullptr, dev_status, stream);
        if (st != Q8_OK) return st;
        launches += last_launch_info().launches;
    }
    last_launch_info().launches = launches;
    return Q8_OK;
}

q8_status q8_linear_wseg(const float *X, const int8_t *Wq, const float *S_w, int64_t w_seg_rows, const float *S_x,
                         const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K, void *workspace,
                         size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc, void *stream)
{
    if (w_seg_rows <= 0) return Q8_ERR_SHAPE;
    if (M > 0 && N > 0 && !Y) return Q8_ERR_NULL;
    return linear_impl(X, Wq, S_w, S_x, bias, act, Y, M, N, K, workspace, workspace_bytes, dbg_Xq, dbg_acc, stream, false,
                       nullptr, nullptr, w_seg_rows);
}

q8_status q8_linear_q_wseg(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w, int64_t w_seg_rows,
                           const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K, int32_t *dbg_acc,
                           int32_t *dev_status, void *stream)
{
    if (w_seg_rows <= 0) return Q8_ERR_SHAPE;
    if (M > 0 && N > 0 && !Y) return Q8_ERR_NULL;
    return linear_q_impl(Xq, S_x, Wq, S_w, bias, act, Y, nullptr, nullptr, M, N, K, dbg_acc, dev_status, stream,
                         w_seg_rows);
}

q8_status q8_linear_requant(const float *X, const int8_t *Wq, const float *S_w, const float *S_x, const float *bias,
                            int act, const float *S_y, int8_t *Yq, float *Y, int64_t M, int64_t N, int64_t K,
                            void *workspace, size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc, void *stream)
{
    if (M > 0 && N > 0 && !Yq) return Q8_ERR_NULL;
    return linear_impl(X, Wq, S_w, S_x, bias, act, Y, M, N, K, workspace, workspace_bytes, dbg_Xq, dbg_acc, stream, false,
                       Yq, S_y);
}

q8_status q8_embedding(const int32_t *ids, int64_t T, const int8_t *Eq, const float *S_e, int64_t V, int64_t H,
                       float *out, int8_t *rows_q, int32_t *dev_status, void *stream)
{
    last_launch_info() = LaunchInfo();
    if (T < 0 || V < 0 || H < 0) return Q8_ERR_SHAPE;
    if (T == 0 || H == 0) return Q8_OK;
    if (!ids || !S_e || !out) return Q8_ERR_NULL;
    if (V > 0 && !Eq) return Q8_ERR_NULL;
    if (V > (int64_t)INT_MAX) return Q8_ERR_SHAPE;
    if (T > (int64_t)LLONG_MAX / H) return Q8_ERR_SHAPE;
    if (!aligned_to(ids, 4) || !aligned_to(S_e, 4) || !aligned_to(out, 4) ||
        (dev_status && !aligned_to(dev_status, 4)))
        return Q8_ERR_ALIGN;
    Q8_CUDA_TRY(launch_embedding(ids, T, Eq, S_e, V, H, out, rows_q, dev_status, static_cast<cudaStream_t>(stream)));
    last_launch_info().launches = 1;
    return Q8_OK;
}

static q8_status add_layernorm_impl(const float *x, const float *r1, const float *r2, const float *gamma,
                                    const float *beta, float eps, int64_t rows, int64_t H, float *out, const float *S_q,
                                    int8_t *out_q, void *stream, uint32_t *amax = nullptr)
{
    last_launch_info() = LaunchInfo();
    if (rows < 0 || H < 0 || H > 12288 || rows > (int64_t)INT_MAX) return Q8_ERR_SHAPE;
    if (rows == 0 || H == 0) return Q8_OK;
    if (!x || (!out && !out_q) || (out_q && !S_q)) return Q8_ERR_NULL;
    if (!(eps >= 0.0f)) return Q8_ERR_ARG;
    if (!aligned_to(x, 4) || !aligned_to(out, 4) || !aligned_to(r1, 4) || !aligned_to(r2, 4) || !aligned_to(gamma, 4) ||
        !aligned_to(beta, 4) || !aligned_to(S_q, 4) || !aligned_to(amax, 4))
        return Q8_ERR_ALIGN;
    Q8_CUDA_TRY(launch_add_layernorm(x, r1, r2, gamma, beta, eps, rows, H, out, S_q, out_q, amax,
                                     static_cast<cudaStream_t>(stream)));
    last_launch_info().launches = 1;
    return Q8_OK;
}

q8_status q8_add_layernorm(const float *x, const float *r1, const float *r2, const float *gamma, const float *beta,
                           float eps, int64_t rows, int64_t H, float *out, void *stream)
{
    if (rows > 0 && H > 0 && !out) return Q8_ERR_NULL;
    return add_layernorm_impl(x, r1, r2, gamma, beta, eps, rows, H, out, nullptr, nullptr, stream);
}

q8_status q8_add_layernorm_quant(const float *x, const float *r1, const float *r2, const float *gamma,
                                 const float *beta, float eps, int64_t rows, int64_t H, float *out, const float *S_q,
                                 int8_t *out_q, void *stream)
{
    if (rows > 0 && H > 0 && !out_q) return Q8_ERR_NULL;
    return add_layernorm_impl(x, r1, r2, gamma, beta, eps, rows, H, out, S_q, out_q, stream);
}

static q8_status attention_impl(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                                int8_t *ctx_q, void *stream, uint32_t *amax = nullptr)
{
    last_launch_info() = LaunchInfo();
    if (B < 0 || S < 0 || heads < 0 || B > 65535 || heads > 65535 || S > (int64_t)INT_MAX) return Q8_ERR_SHAPE;
    if (B == 0 || S == 0 || heads == 0) return Q8_OK;
    if (!qkv || (!ctx && !ctx_q) || (ctx_q && !S_q)) return Q8_ERR_NULL;
    if (!aligned_to(qkv, 8) || !aligned_to(ctx, 8) || !aligned_to(S_q, 4) || !aligned_to(amax, 4))
        return Q8_ERR_ALIGN;  // 8-byte vector accesses
    Q8_CUDA_TRY(launch_attention(qkv, B, S, heads, ctx, S_q, ctx_q, amax, static_cast<cudaStream_t>(stream)));
    last_launch_info().launches = 1;
    return Q8_OK;
}

q8_status q8_attention(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, void *stream)
{
    if (B > 0 && S > 0 && heads > 0 && !ctx) return Q8_ERR_NULL;
    return attention_impl(qkv, B, S, heads, ctx, nullptr, nullptr, stream);
}

q8_status q8_attention_quant(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                             int8_t *ctx_q, void *stream)
{
    if (B > 0 && S > 0 && heads > 0 && !ctx_q) return Q8_ERR_NULL;
    return attention_impl(qkv, B, S, heads, ctx, S_q, ctx_q, stream);
}

q8_status q8_add_layernorm_absmax(const float *x, const float *r1, const float *r2, const float *gamma,
                                  const float *beta, float eps, int64_t rows, int64_t H, float *out,
                                  uint32_t *absmax_bits, void *stream)
{
    if (!absmax_bits || (rows > 0 && H > 0 && !out)) return Q8_ERR_NULL;
    return add_layernorm_impl(x, r1, r2, gamma, beta, eps, rows, H, out, nullptr, nullptr, stream, absmax_bits);
}

q8_status q8_attention_absmax(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, uint32_t *absmax_bits,
                              void *stream)
{
    if (!absmax_bits || (B > 0 && S > 0 && heads > 0 && !ctx)) return Q8_ERR_NULL;
    return attention_impl(qkv, B, S, heads, ctx, nullptr, nullptr, stream, absmax_bits);
}

q8_status q8_linear_dyn(const float *X, const uint32_t *x_absmax, const int8_t *Wq, const float *S_w, const float *bias,
                        int act, float *Y, uint32_t *y_absmax, int64_t M, int64_t N, int64_t K, void *workspace,
                        size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc, void *stream)
{
    if (M > 0 && N > 0 && (!Y || !x_absmax)) return Q8_ERR_NULL;
    return linear_impl(X, Wq, S_w, nullptr, bias, act, Y, M, N, K, workspace, workspace_bytes, dbg_Xq, dbg_acc, stream,
                       false, nullptr, nullptr, 0, x_absmax, y_absmax);
}

q8_status q8_poll_status(void *dev_status, uint32_t *raw_bits, void *stream)
{
    if (!dev_status) return Q8_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t bits = 0;
    Q8_CUDA_TRY(cudaMemcpyAsync(&bits, dev_status, sizeof(bits), cudaMemcpyDeviceToHost, s));
    Q8_CUDA_TRY(cudaMemsetAsync(dev_status, 0, sizeof(bits), s));
    Q8_CUDA_TRY(cudaStreamSynchronize(s));
    if (raw_bits) *raw_bits = bits;
    for (int code = 1; code < 32; ++code)
        if (bits & (1u << code)) return static_cast<q8_status>(code);
    return Q8_OK;
}

const char *q8_status_string(q8_status s)
{
    switch (s) {
        case Q8_OK: return "ok";
        case Q8_ERR_NULL: return "required pointer is NULL";
        case Q8_ERR_SHAPE: return "invalid or unsupported shape";
        case Q8_ERR_ALIGN: return "pointer misaligned";
        case Q8_ERR_SCALE: return "max|x| was zero or non-finite; scale forced to 1";
        case Q8_ERR_INDEX: return "embedding id out of range";
        case Q8_ERR_OVERFLOW: return "K too large for an exact Int32 accumulator";
        case Q8_ERR_WORKSPACE: return "workspace too small";
        case Q8_ERR_TIMEOUT: return "bounded device wait expired";
        case Q8_ERR_CUDA: return "CUDA call failed";
        case Q8_ERR_ARG: return "invalid argument value";
    }
    return "unknown status";
}

void q8_last_launch_info(int *gemm_kernel, int *launches, int *block_n, int *grid, int *ctas)
{
    const LaunchInfo &li = last_launch_info();
    if (gemm_kernel) *gemm_kernel = li.gemm_kernel;
    if (launches) *launches = li.launches;
    if (block_n) *block_n = li.block_n;
    if (grid) *grid = li.grid;
    if (ctas) *ctas = li.ctas;
}

q8_status q8_tune_gemm_tile(int block_n, int ctas)
{
    const bool automatic = block_n == 0 && ctas == 0;
    const bool single = ctas == 1 && (block_n == 32 || block_n == 64 || block_n == 128 || block_n == 256);
    const bool pair = ctas == 2 && block_n == 256;
    if (!automatic && !single && !pair) return Q8_ERR_ARG;
    set_gemm_tile_override(block_n, ctas);
    return Q8_OK;
}

q8_status q8_tune_gemm_epilogue_warps(int warps)
{
    if (warps != 0 && warps != 8 && warps != 16) return Q8_ERR_ARG;
    set_gemm_epilogue_warps(warps);
    return Q8_OK;
}

void q8_tune_attention(int use_tensor_cores) { set_attention_tensor_cores(use_tensor_cores != 0); }

q8_status q8_attention_status_word(void **dev_status)
{
    if (dev_status == nullptr) return Q8_ERR_NULL;
    *dev_status = attention_status_word();
    return *dev_status != nullptr ? Q8_OK : Q8_ERR_CUDA;
}

void q8_tune_gemm_tail_split(int enable) { set_gemm_tail_split(enable != 0); }
void q8_tune_gemm_direct_store(int mode) { set_gemm_direct_store(mode); }

int q8_last_launch_tail_split(void) { return last_launch_info().tail_split; }
int q8_last_launch_store_mode(void) { return last_launch_info().store_mode; }

}  // extern "C"
