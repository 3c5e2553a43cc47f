/*
 * q8.h -- C ABI of the sm_100a int8 inference path of Q8BERT (arXiv 1910.06188).
 *
 * The library implements the inference mode of the paper's quantised layers (Sec. 3):
 * symmetric linear quantisation to Int8 (Eq. 1, Eq. 2), per-tensor weight scale (Eq. 3),
 * activation scale from an EMA of max|x| (Eq. 4) or computed per incoming tensor (Sec. 4.1),
 * the Int8 x Int8 -> Int32 GEMM accumulated onto an Int32 bias, and the Int8 embedding lookup.
 *
 * Conventions that hold for every entry point
 *   - All data pointers are DEVICE pointers on the current CUDA device unless a parameter says
 *     "host".  The caller owns every buffer; the library never allocates or frees device memory.
 *   - Tensors are dense row-major.  Activations X are [M, K], weights W / W_q are [N, K]
 *     (out-features first, so Y = X W^T + b), outputs Y are [M, N].
 *   - Scales are single fp32 values living in device memory, so no call forces a host sync.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue
 *     work; they return after argument checks and launches.
 *   - Argument errors are returned at once as a q8_status and nothing is launched.  Conditions
 *     only the device can see (zero or non-finite max|x|, an out-of-range token id, a bounded
 *     device-side wait that ran out) are OR-ed as bit (1 << code) into a device status word and
 *     read back with q8_poll_status().  No kernel traps or spins without limit.
 *   - float pointers must be 4-byte aligned; 16-byte alignment of X, Y, W_q (and K % 16 == 0)
 *     selects the vectorised / tensor-core kernels, anything else runs the generic kernels
 *     with identical results.
 *   - Results are deterministic: the same inputs give bit-identical outputs.
 *
 * Tuning hooks, measurement aids and the wait self-test live in q8_tools.h (same library); nothing in this header
 * depends on them.
 */
#ifndef Q8_H_
#define Q8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    Q8_OK = 0,
    Q8_ERR_NULL = 1,      /* a required pointer is NULL */
    Q8_ERR_SHAPE = 2,     /* negative size, K == 0, size beyond the supported range */
    Q8_ERR_ALIGN = 3,     /* pointer not aligned to its element type / workspace not 256-byte aligned */
    Q8_ERR_SCALE = 4,     /* device: max|x| was 0 or non-finite; scale forced to 1 */
    Q8_ERR_INDEX = 5,     /* device: embedding id outside [0, V); that row is written as zeros */
    Q8_ERR_OVERFLOW = 6,  /* K > 133144: K * 127^2 would not fit the Int32 accumulator */
    Q8_ERR_WORKSPACE = 7, /* workspace smaller than q8_linear_workspace_bytes() */
    Q8_ERR_TIMEOUT = 8,   /* device: a bounded wait inside the GEMM kernel expired */
    Q8_ERR_CUDA = 9,      /* a CUDA runtime / driver call failed */
    Q8_ERR_ARG = 10       /* invalid enum or parameter value (act, decay) */
} q8_status;

/* Largest reduction length for which the Int32 accumulator is exact: floor((2^31-1)/127^2). */
#define Q8_MAX_K 133144

/* Activation applied after dequantisation (Sec. 3 keeps GELU in FP32). */
#define Q8_ACT_NONE 0
#define Q8_ACT_GELU 1 /* y * Phi(y), erf form */

/* Eq. 3 followed by Eq. 1 (one-time weight preparation; also used for embedding tables).
 *   W      [N, K] fp32, read.
 *   Wq     [N, K] int8, written: Clamp(nint(W * S_w), -127, 127).
 *   S_w    1 fp32, written: 127 / max|W|  (1.0 and Q8_ERR_SCALE flagged if max|W| is 0 / non-finite).
 *   dev_status  optional device status word (may be NULL), OR-ed into, never cleared.
 * N == 0 or K == 0 is a no-op that writes S_w = 1. */
q8_status q8_quantize_weight(const float *W, int64_t N, int64_t K, int8_t *Wq, float *S_w,
                             int32_t *dev_status, void *stream);

/* Eq. 1 on an activation tensor (flat, `numel` elements).
 *   S_x != NULL: static scale (an Eq. 4 result), read.           S_x_used may be NULL.
 *                A value that is not a positive finite number flags Q8_ERR_SCALE in dev_status.
 *   S_x == NULL: dynamic scale of Sec. 4.1, S = 127 / max|X| over this tensor, written to
 *                S_x_used (required; it also serves as the reduction scratch word).
 *   Xq     int8 [numel], written. */
q8_status q8_quantize_activation(const float *X, int64_t numel, const float *S_x, int8_t *Xq,
                                 float *S_x_used, int32_t *dev_status, void *stream);

/* Eq. 4: one calibration batch.  `state` is a q8_calibrate_state_bytes()-byte, 16-byte aligned,
 * zero-initialised device block laid out as
 *   { float ema; float S_x; int32 n_batches; uint32 scratch; int32 status; int32 pad[3]; }
 * The first batch sets ema = max|X|; later ones do ema += (1 - decay) * (max|X| - ema) in fp32;
 * then S_x = 127 / ema.  decay must lie in [0, 1); decay 0 keeps no history: ema is exactly this batch's
 * max|X| and S_x exactly the dynamic scale of Sec. 4.1.  A batch with numel == 0 carries no observation and
 * leaves the state untouched (nothing is launched).  &state->S_x can be passed as S_x to q8_linear. */
q8_status q8_calibrate(const float *X, int64_t numel, float decay, void *state, void *stream);
size_t q8_calibrate_state_bytes(void);

/* Training-mode building blocks (Sec. 2.2 and the training sentence of Sec. 3).
 * q8_fake_quantize: Xhat = Quantize(X | S) / S, the rounding of Eq. 1 simulated in fp32 (X, Xhat flat fp32 of
 *   `numel` elements, may alias; S a device scalar, e.g. &state->S_x kept current by q8_calibrate, which is the
 *   EMA update of Eq. 4 that training performs on every forward).
 * q8_ste_backward: the straight-through estimator of Eq. 5, d Xhat / d X = 1: grad_in = grad_out (a device copy;
 *   a no-op when the two pointers are equal). */
q8_status q8_fake_quantize(const float *X, int64_t numel, const float *S, float *Xhat, void *stream);
q8_status q8_ste_backward(const float *grad_out, int64_t numel, float *grad_in, void *stream);

/* The quantised fully-connected layer in inference mode (Sec. 3):
 *   X_q = Quantize(X | S_x)  (Eq. 1);  acc = X_q W_q^T in Int32, accumulated onto the Int32 bias
 *   b_q = Clamp(nint(b * fl32(S_x * S_w)), -(2^31-1), 2^31-1);  Y = (acc + b_q) / (S_x * S_w);
 *   optional GELU.
 *   X [M,K] fp32; Wq [N,K] int8 with its scale S_w (from q8_quantize_weight); bias [N] fp32 or NULL.
 *   S_x: static activation scale, or NULL for the dynamic scale 127 / max|X| of Sec. 4.1.  A static scale
 *     that is not a positive finite number flags Q8_ERR_SCALE in the status word (the output is then meaningless).
 *   act: Q8_ACT_NONE or Q8_ACT_GELU.      Y [M,N] fp32, written.
 *   workspace: >= q8_linear_workspace_bytes(M,N,K) bytes, 256-byte aligned, caller-owned scratch
 *     (status word at offset 0, then the quantised activation).  Its contents need not be
 *     initialised; the status word is cleared at the start of every call.  Two calls that share
 *     a workspace must be ordered on the stream.
 *   dbg_Xq [M,K] int8 / dbg_acc [M,N] int32: optional (NULL to skip) copies of the quantised
 *     activation and of acc + b_q, for bit-exact checks.
 * M == 0 or N == 0 is a no-op.  K == 0 is Q8_ERR_SHAPE; K > Q8_MAX_K is Q8_ERR_OVERFLOW. */
q8_status q8_linear(const float *X, const int8_t *Wq, const float *S_w, const float *S_x,
                    const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K,
                    void *workspace, size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc,
                    void *stream);
size_t q8_linear_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Same layer on an activation that is already Int8 (the GEMM, bias, dequantise and activation
 * steps only).  Xq [M,K] int8 and S_x (required) describe the quantised input.  dev_status is an
 * optional status word that receives Q8_ERR_TIMEOUT. */
q8_status q8_linear_q(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w,
                      const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K,
                      int32_t *dbg_acc, int32_t *dev_status, void *stream);

/* q8_linear / q8_linear_q forced onto the generic (any shape, any alignment, CUDA-core) GEMM
 * kernel that q8_linear uses by itself when K % 16 != 0 or an operand is not 16-byte aligned.
 * Same arguments, same results; kept public as an on-device cross-check of the tensor-core kernel. */
q8_status q8_linear_generic(const float *X, const int8_t *Wq, const float *S_w, const float *S_x,
                            const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K,
                            void *workspace, size_t workspace_bytes, int8_t *dbg_Xq,
                            int32_t *dbg_acc, void *stream);

/* q8_linear for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a deployment convenience, not part of the method.)
 * Intended for code that runs where cudaMalloc is off limits: a serving loop whose memory was
 * partitioned at start-up, a plugin working inside an engine that owns all allocations, a process
 * whose allocator is frozen after initialisation.  It computes exactly what q8_linear computes, with
 * the same arguments minus the workspace: the scratch (status word + Int8 activation) is a fixed
 * array inside the library image, present on every GPU that loads the library until the process
 * exits.  Once the library is warm on a device the call performs no allocation of any kind; the very
 * first call on a device (and the first use of each GEMM tile configuration) makes the CUDA runtime load
 * the kernels and the array there, so issue one warm-up call per device and shape class at start-up.
 * The looked-up addresses are cached per device and do not survive cudaDeviceReset.
 *   Limit: M * K <= Q8_NOALLOC_MAX_MK (16 Mi elements, i.e. 16 MiB of scratch + a 256-byte header);
 *     larger activations are refused with Q8_ERR_WORKSPACE before anything is launched.
 *   status_word (host pointer, may be NULL) receives the device address of the status word, which
 *     can be handed to q8_poll_status.
 *   The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   Every call on a device uses the same array: calls that may overlap on the GPU (different
 *     streams without ordering, or host threads) race on it.  Order them, or use q8_linear with
 *     separate workspaces.  The header words are cleared at the start of each call; the rest is
 *     simply overwritten. */
#define Q8_NOALLOC_MAX_MK (16 * 1024 * 1024)
q8_status q8_linear_noalloc(const float *X, const int8_t *Wq, const float *S_w, const float *S_x,
                            const float *bias, int act, float *Y, int64_t M, int64_t N, int64_t K,
                            int8_t *dbg_Xq, int32_t *dbg_acc, void **status_word, void *stream);

/* Quantised embedding layer in inference mode (Sec. 3): gathers Int8 rows of the table and hands
 * them to the FP32 consumer dequantised: out[t, :] = Eq[ids[t], :] / S_e.
 *   ids [T] int32; Eq [V,H] int8; S_e 1 fp32; out [T,H] fp32 (written); rows_q [T,H] int8 optional
 *   raw-row output (NULL to skip).  An id outside [0,V) yields a zero row and flags Q8_ERR_INDEX
 *   in dev_status (optional). */
q8_status q8_embedding(const int32_t *ids, int64_t T, const int8_t *Eq, const float *S_e, int64_t V,
                       int64_t H, float *out, int8_t *rows_q, int32_t *dev_status, void *stream);

/* FP32 support operations of the BERT encoder.  Sec. 3 keeps Softmax, Layer Normalization and GELU
 * in FP32, and the attention score / context products are not FC layers, so they are not quantised;
 * these two calls let a whole encoder forward run through this library.
 *
 * out[r, :] = LayerNorm(x[r, :] + r1[r, :] + r2[r, :]) * gamma + beta   (rows x H, row-major fp32;
 * r1, r2, gamma, beta may be NULL: no residual / gamma 1 / beta 0; mean and variance over H, biased
 * variance, eps inside the square root).  H <= 12288.  out may alias x, r1 or r2. */
q8_status q8_add_layernorm(const float *x, const float *r1, const float *r2, const float *gamma,
                           const float *beta, float eps, int64_t rows, int64_t H, float *out, void *stream);

/* Multi-head self-attention without mask, head dimension 64, fp32:
 *   qkv [B*S, 3*H] = [q | k | v] per token (H = heads * 64), ctx [B*S, H] (written):
 *   ctx[b, i, h*64 : h*64+64] = sum_j softmax_j(q_i . k_j / 8) v_j  over the S tokens of sequence b. */
q8_status q8_attention(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx, void *stream);

/* Weight scales per block of output rows.  Eq. 3 gives every FC layer of the paper its own S_w; when several
 * layers that share an input are stored as one matrix (the fused QKV projection: three layers of H rows each),
 * one scale per block of `seg_rows` rows keeps exactly the paper's per-layer scales: the result equals running
 * the blocks as separate quantised FC layers.  S_w is then an array of ceil(N / seg_rows) device floats.
 * The tensor-core kernel needs seg_rows % 32 == 0; other values run the generic kernel. */
q8_status q8_quantize_weight_segments(const float *W, int64_t N, int64_t K, int64_t seg_rows, int8_t *Wq,
                                      float *S_w, int32_t *dev_status, void *stream);
q8_status q8_linear_wseg(const float *X, const int8_t *Wq, const float *S_w, int64_t w_seg_rows,
                         const float *S_x, const float *bias, int act, float *Y, int64_t M, int64_t N,
                         int64_t K, void *workspace, size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc,
                         void *stream);
q8_status q8_linear_q_wseg(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w,
                           int64_t w_seg_rows, const float *bias, int act, float *Y, int64_t M, int64_t N,
                           int64_t K, int32_t *dbg_acc, int32_t *dev_status, void *stream);

/* Fused re-quantisation (Sec. 3 inference mode chained layer to layer; Eq. 1 with the consumer's Eq. 4
 * scale): the producer of an activation also emits it as Int8 at the NEXT quantised layer's static
 * scale S_y / S_q, so that layer can run q8_linear_q with no separate quantise pass and, for FFN1, no
 * fp32 round trip through HBM.  The Int8 values equal Quantize(y | S) of the very fp32 value the plain
 * call would have stored.  The fp32 output pointer (Y / out / ctx) may be NULL when only Int8 is wanted.
 * Other arguments are as in q8_linear, q8_linear_q, q8_add_layernorm and q8_attention. */
q8_status q8_linear_requant(const float *X, const int8_t *Wq, const float *S_w, const float *S_x,
                            const float *bias, int act, const float *S_y, int8_t *Yq, float *Y, int64_t M,
                            int64_t N, int64_t K, void *workspace, size_t workspace_bytes, int8_t *dbg_Xq,
                            int32_t *dbg_acc, void *stream);
q8_status q8_linear_q_requant(const int8_t *Xq, const float *S_x, const int8_t *Wq, const float *S_w,
                              const float *bias, int act, const float *S_y, int8_t *Yq, float *Y, int64_t M,
                              int64_t N, int64_t K, int32_t *dbg_acc, int32_t *dev_status, void *stream);
q8_status q8_add_layernorm_quant(const float *x, const float *r1, const float *r2, const float *gamma,
                                 const float *beta, float eps, int64_t rows, int64_t H, float *out,
                                 const float *S_q, int8_t *out_q, void *stream);
q8_status q8_attention_quant(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx,
                             const float *S_q, int8_t *ctx_q, void *stream);

/* Dynamic quantisation without stand-alone abs-max passes (Sec. 4.1: the scale 127 / max|x| is computed for every
 * incoming activation tensor).  The kernel that PRODUCES an activation can fold max|y| of what it stores into a
 * caller-owned device word while it writes it, and the quantised layer that consumes the activation takes its
 * dynamic scale from that word instead of reading the whole tensor once more:
 *   absmax_bits / y_absmax: device uint32 holding the IEEE bits of a non-negative fp32 (0 before the producer runs:
 *     the caller clears it; producers only ever raise it, with an atomic max, so several producers may share a word
 *     when their union is the tensor).  NaN outputs are skipped, an infinite output makes the word +Inf.
 *   q8_add_layernorm_absmax / q8_attention_absmax: q8_add_layernorm / q8_attention plus that word.
 *   q8_linear_dyn: q8_linear with the dynamic scale S_x = 127 / float(*x_absmax) (required; the word must be final,
 *     i.e. its producer ordered before this call on the stream); S_x is left in the workspace header as in q8_linear,
 *     Q8_ERR_SCALE is flagged there when the word is 0 or +Inf.  y_absmax (may be NULL) receives max|Y| of this
 *     layer's own output (after GELU when act says so) for the next dynamically quantised layer.
 * The results are bit-identical to q8_add_layernorm, q8_attention and q8_linear with S_x == NULL. */
q8_status q8_add_layernorm_absmax(const float *x, const float *r1, const float *r2, const float *gamma,
                                  const float *beta, float eps, int64_t rows, int64_t H, float *out,
                                  uint32_t *absmax_bits, void *stream);
q8_status q8_attention_absmax(const float *qkv, int64_t B, int64_t S, int64_t heads, float *ctx,
                              uint32_t *absmax_bits, void *stream);
q8_status q8_linear_dyn(const float *X, const uint32_t *x_absmax, const int8_t *Wq, const float *S_w,
                        const float *bias, int act, float *Y, uint32_t *y_absmax, int64_t M, int64_t N, int64_t K,
                        void *workspace, size_t workspace_bytes, int8_t *dbg_Xq, int32_t *dbg_acc, void *stream);

/* Synchronises `stream`, reads the device status word at `dev_status` (a q8_linear workspace
 * pointer works: the word sits at offset 0), clears it, and returns the lowest-numbered code
 * whose bit was set (Q8_OK if none).  `raw_bits` (host pointer, may be NULL) receives the word. */
q8_status q8_poll_status(void *dev_status, uint32_t *raw_bits, void *stream);

const char *q8_status_string(q8_status s);

/* What the most recent call on this host thread enqueued: which GEMM kernel it chose (0 none,
 * 1 tcgen05, 2 generic), how many kernels it launched, the tile width, the grid size and how many
 * CTAs share one tile (2 = cta_group::2 pairs).  Host-side bookkeeping for benchmarks and tests;
 * any pointer may be NULL. */
void q8_last_launch_info(int *gemm_kernel, int *launches, int *block_n, int *grid, int *ctas);

/* q8_attention / q8_attention_quant run on the tensor cores when the padded sequence fits the accumulator
 * memory (S rounded up to a multiple of 64, plus 64, at most 512 columns: S <= 448) and the pointers are
 * 16-byte aligned: both products as tcgen05.mma kind::tf32 on operands split into a TF32-exact high part and a
 * low remainder, three partial products accumulated in fp32, which keeps fp32-grade accuracy.  Otherwise a
 * CUDA-core fp32 kernel computes the same thing.  The tensor-core kernel bounds
 * its waits; a time-out sets the Q8_ERR_TIMEOUT bit in a per-device status word whose device address
 * q8_attention_status_word returns (poll it with q8_poll_status). */
q8_status q8_attention_status_word(void **dev_status);

#ifdef __cplusplus
}
#endif
#endif /* Q8_H_ */
