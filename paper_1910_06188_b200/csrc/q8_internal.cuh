// Internal declarations shared by the translation units of libq8 (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "q8.h"
#include "q8_tools.h"

namespace q8 {

// Layout of the head of a q8_linear workspace.
struct WorkspaceHeader {
    int32_t status;        // OR of (1 << q8_status) bits raised by kernels
    float S_x_dyn;         // dynamic mode: 127 / max|X|, written by the quantise kernel
    uint32_t absmax_bits;  // dynamic mode: float bits of max|X| (atomicMax scratch, zero at the start of a call)
    int32_t pad;
};
constexpr size_t kWorkspaceHeaderBytes = 256;

// Device block behind q8_calibrate (Eq. 4 running state).
struct CalibState {
    float ema;
    float S_x;
    int32_t n_batches;
    uint32_t scratch_bits;
    int32_t status;
    int32_t pad[3];
};

struct GemmArgs {
    const int8_t *Xq;   // [M,K]
    const int8_t *Wq;   // [N,K]
    const float *S_x;   // device scalar
    const float *S_w;   // device scalar, or one scale per block of w_seg output rows of W
    int64_t w_seg = 0;  // rows of W (output features) that share one weight scale; 0 = one scale for all
    const float *bias;  // [N] or nullptr
    float *Y;           // [M,N] fp32 output, or nullptr when only the re-quantised output is wanted
    int8_t *Yq;         // [M,N] Int8 output Quantize(y | S_y) (Eq. 1 at the consumer's scale), or nullptr
    const float *S_y;   // device scalar, required with Yq
    int32_t *dbg_acc;   // [M,N] or nullptr
    uint32_t *y_absmax = nullptr;  // optional: max|y| over the stored output is folded into this word (float bits, atomicMax)
    int32_t *status;    // device status word or nullptr
    int64_t M, N, K;
    int act;
};

struct LaunchInfo {
    int gemm_kernel = 0;  // 0 none, 1 tcgen05, 2 generic
    int launches = 0;
    int block_n = 0;
    int ctas = 0;  // CTAs cooperating on one tile (1, or 2 for cta_group::2)
    int epilogue_warps = 0;
    int grid = 0;
    int tail_split = 1;  // tiles of the last scheduling round cut into this many narrower ones
    int store_mode = 0;  // fp32 output of the tcgen05 GEMM: 0 stored by the lanes, 1 staged + TMA store, 2 unstaged
};
LaunchInfo &last_launch_info();

// ---- elementwise / reduction launchers (q8_elementwise.cu) ----
// max|x| folded into *bits (must hold 0 or an earlier maximum) with atomicMax on the float bits.
cudaError_t launch_absmax(const float *x, int64_t n, uint32_t *bits, cudaStream_t s);
// *S = 127 / float(*bits) in place (bits and S may alias); flags Q8_ERR_SCALE on 0 / non-finite.
cudaError_t launch_scale_from_absmax(const uint32_t *bits, float *S, int32_t *status, cudaStream_t s);
// clear_word (may be NULL): a device word the kernel sets to zero before anything else (a call's status word).
// A scale *S that is not a positive finite number raises Q8_ERR_SCALE in *status (or, without one, in *clear_word).
cudaError_t launch_quantize(const float *x, int64_t n, const float *S, int8_t *xq, int8_t *xq_copy,
                            cudaStream_t s, int32_t *clear_word = nullptr, int32_t *status = nullptr);
// Eq. 1 with S = 127 / float(*absmax_bits) derived inside the kernel (dynamic scale); *S_out receives S and
// *status the Q8_ERR_SCALE bit when the maximum is 0 or not finite (S = 1 then).  absmax_bits and S_out differ.
// clear_status: start *status at zero first (the call's status word, when no memset precedes the kernel).
cudaError_t launch_quantize_dynamic(const float *x, int64_t n, const uint32_t *absmax_bits, float *S_out,
                                    int32_t *status, int8_t *xq, int8_t *xq_copy, cudaStream_t s,
                                    bool clear_status = false);
// Small tensors (n <= 196608, n % 4 == 0, 16-byte aligned): abs-max, scale and Eq. 1 in one launch of one cluster.
// *status (may be NULL) is SET (0 or the Q8_ERR_SCALE bit), not OR-ed into.
bool quantize_dynamic_small_supported(const float *x, int64_t n, const int8_t *xq, const int8_t *xq_copy);
cudaError_t launch_quantize_dynamic_small(const float *x, int64_t n, float *S_out, int32_t *status, int8_t *xq,
                                          int8_t *xq_copy, cudaStream_t s);
cudaError_t launch_ema_update(CalibState *st, float decay, cudaStream_t s);
cudaError_t launch_fake_quantize(const float *x, int64_t n, const float *S, float *xhat, cudaStream_t s);
cudaError_t launch_embedding(const int32_t *ids, int64_t T, const int8_t *Eq, const float *S_e, int64_t V,
                             int64_t H, float *out, int8_t *rows_q, int32_t *status, cudaStream_t s);

// ---- fp32 encoder support (q8_support.cu) ----
// amax (may be NULL): max|output| is folded into this device word (float bits, atomicMax; it must hold 0 or an
// earlier maximum), so that a dynamically quantised consumer (Sec. 4.1) needs no abs-max pass of its own.
cudaError_t launch_add_layernorm(const float *x, const float *r1, const float *r2, const float *gamma,
                                 const float *beta, float eps, int64_t rows, int64_t H, float *out, const float *S_q,
                                 int8_t *out_q, uint32_t *amax, cudaStream_t s);
cudaError_t launch_attention(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                             int8_t *ctx_q, uint32_t *amax, cudaStream_t s);

// Tensor-core attention (q8_attention_sm100.cu): 3 x TF32 split products with fp32 accumulation in TMEM.
bool attention_tc_supported(const float *qkv, int64_t S, int64_t heads, const float *ctx, const int8_t *ctx_q);
cudaError_t launch_attention_tc(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, const float *S_q,
                                int8_t *ctx_q, uint32_t *amax, cudaStream_t s);
void set_attention_tensor_cores(bool enable);
int32_t *attention_status_word();  // device word that receives Q8_ERR_TIMEOUT from the tensor-core attention kernel

// ---- GEMM launchers ----
bool tcgen05_gemm_supported(const GemmArgs &a);
void set_gemm_tile_override(int block_n, int ctas, int epilogue_warps = 0);  // 0, 0 = automatic choice
void set_gemm_tail_split(bool enable);
void set_gemm_direct_store(int mode);
void set_gemm_epilogue_warps(int warps);  // 0 automatic, 8 or 16
cudaError_t launch_gemm_tcgen05(const GemmArgs &a, cudaStream_t s);  // q8_gemm_sm100.cu
cudaError_t launch_gemm_generic(const GemmArgs &a, cudaStream_t s);  // q8_gemm_generic.cu


// The body of q8_linear / q8_linear_generic: validates, quantises X into `workspace`, runs the GEMM (q8_api.cu).
q8_status linear_impl(const float *X, const int8_t *Wq, const float *S_w, const float *S_x, const float *bias, int act,
                      float *Y, int64_t M, int64_t N, int64_t K, void *workspace, size_t workspace_bytes,
                      int8_t *dbg_Xq, int32_t *dbg_acc, void *stream, bool force_generic, int8_t *Yq = nullptr,
                      const float *S_y = nullptr, int64_t w_seg = 0, const uint32_t *x_absmax = nullptr,
                      uint32_t *y_absmax = nullptr);

// ---- programmatic dependent launch
// A kernel launched with launch_overlapping_tail() may be scheduled while the kernel before it in the stream is
// still draining (its last CTAs finishing), so that its own start-up overlaps that tail.  Such a kernel must call
// grid_dependency_wait() before its first global-memory access: the call returns once the preceding kernel has
// completed and its writes are visible (and at once when the kernel was launched the ordinary way).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the NEXT kernel in the stream (if it was launched with launch_overlapping_tail) be scheduled as soon as every
// CTA of this grid has started, instead of when the last one exits: its CTAs then sit resident, parked in their own
// grid_dependency_wait(), and start the moment this grid has completed.  It does not weaken any ordering: the next
// kernel still touches global memory only after its wait, i.e. after this whole grid has finished.  Kernels call it
// only for SMALL problems (`small`, a grid-uniform condition), where launch latency is a visible share of the run
// time: a BERT-Base forward (32 x 128 tokens) replayed from a graph goes from 1.39 to 1.34 ms; on large problems
// the parked CTAs only get in the way (the M = 24576 FC step went from 505 to 528 us), so those keep the default.
__device__ __forceinline__ void grid_dependency_release_next(bool small)
{
    if (small) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
constexpr int64_t kSmallProblemElems = int64_t(16) << 20;  // elementwise kernels: up to 16 Mi elements count as small

template <typename... KArgs, typename... Args>
cudaError_t launch_overlapping_tail(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Eq. 1 on one value: one rounded fp32 multiply, nearest-even integer (NaN -> 0, saturating), symmetric clamp.
__device__ __forceinline__ int32_t quantize_value(float x, float S)
{
    int32_t q = __float2int_rn(__fmul_rn(x, S));
    return max(-127, min(127, q));
}

// Four values of Eq. 1 packed little-endian (a in the lowest byte).  The lower clamp is an integer max; the upper
// clamp and the packing are done by cvt.pack.sat.s8.s32, which saturates each Int32 to [-128, 127] while it packs
// two of them into the low half of the result and moves the low half of its third operand into the high half.
__device__ __forceinline__ uint32_t quantize_pack4(float a, float b, float c, float d, float S)
{
    const int32_t qa = max(__float2int_rn(__fmul_rn(a, S)), -127), qb = max(__float2int_rn(__fmul_rn(b, S)), -127);
    const int32_t qc = max(__float2int_rn(__fmul_rn(c, S)), -127), qd = max(__float2int_rn(__fmul_rn(d, S)), -127);
    uint32_t hi, r;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(qd), "r"(qc), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(qb), "r"(qa), "r"(hi));
    return r;
}

// ---- epilogue arithmetic shared by both GEMM kernels ----
// Bias quantised at the product scale: Clamp(nint(b * S_out), -(2^31-1), 2^31-1).
__device__ __forceinline__ int32_t quantize_bias(float b, float S_out)
{
    // cvt.rni saturates at the int32 range and maps NaN to 0; only INT_MIN needs the symmetric clamp.
    int32_t q = __float2int_rn(__fmul_rn(b, S_out));
    return max(q, -2147483647);
}

__device__ __forceinline__ float gelu_erf(float y)
{
    return 0.5f * y * (1.0f + erff(y * 0.70710678118654752440f));
}

// acc + b_q in Int32 (two's-complement wrap), dequantised with the reciprocal of the product scale.
__device__ __forceinline__ float finish_output(int32_t acc_plus_bias, float inv_S_out, int act)
{
    float y = __fmul_rn(__int2float_rn(acc_plus_bias), inv_S_out);
    return act == Q8_ACT_GELU ? gelu_erf(y) : y;
}

// Folds a warp's running max|.| into a device word: non-negative floats order like their bit patterns, NaN never
// enters (fmaxf drops it), +Inf propagates; nothing is written for an all-zero warp.
__device__ __forceinline__ void warp_fold_absmax(float m, uint32_t *word)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m > 0.0f) atomicMax(word, __float_as_uint(m));
}

__device__ __forceinline__ int32_t add_wrap(int32_t a, int32_t b)
{
    return (int32_t)((uint32_t)a + (uint32_t)b);
}

}  // namespace q8
