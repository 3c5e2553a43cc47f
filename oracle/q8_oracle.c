/*
 * q8_oracle.c -- slow, plain CPU restatement of Q8BERT's 8-bit inference arithmetic.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker that the CUDA library is compared
 * against.  It shares no code, header, table or constant with the CUDA path and nothing on the
 * product path may call it.  Every function follows the paper's steps in the paper's order with
 * no blocking, fusion or reordering; OpenMP only splits the outermost independent loop.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC q8_oracle.c -lm
 * (-ffp-contract=off matters: the quantiser's product x*S must be ONE rounded fp32 multiply.)
 *
 * Precision: the quantiser (Eq. 1-4) decides integers, so it is evaluated in IEEE fp32 exactly
 * as defined below (the precision both sides agree on); everything after the integer
 * accumulator (dequantise, GELU, embedding dequantise) is evaluated in fp64.
 *
 * Readings of points the paper leaves open (each one is also listed in the design notes):
 *   - the nearest-integer bracket of Eq. 1 rounds halves to even (IEEE default rounding);
 *   - x*S is one fp32 multiply, rounded to nearest even, before the nearest-integer step;
 *   - max|x| == 0 or non-finite  =>  scale 1.0 and a flag (Eq. 3/4 would divide by zero);
 *   - NaN quantises to 0, +-Inf to +-M (follows from Clamp once NaN is mapped to 0);
 *   - EMA: first observation initialises, then ema += (1-d)*(m-ema), each op rounded in fp32;
 *   - bias: b_q = Clamp(nint(b * fl32(S_x*S_w)), -M(32), M(32)) as int32 (Sec. 3, inference mode);
 *   - dequantise: y = (acc + b_q) / (S_x*S_w) (inverse of Eq. 1; never printed in the paper);
 *   - GELU is the erf form 0.5*y*(1+erf(y/sqrt 2)) (Sec. 3 only names GELU).
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>

/* Eq. 2: M = 2^(b-1) - 1, the largest quantised magnitude for b bits. */
int64_t q8o_M(int b)
{
    return ((int64_t)1 << (b - 1)) - 1;
}

/* max|t_i| over a tensor (the quantity inside Eq. 3 and Eq. 4).  NaN entries are skipped;
 * an infinite entry makes the result infinite (the caller then flags the scale). */
float q8o_absmax(const float *t, int64_t n)
{
    float m = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        float a = fabsf(t[i]);
        if (a > m) m = a;            /* false for NaN, so NaN is skipped */
    }
    return m;
}

/* Eq. 3 (weights) and its Sec. 4.1 reuse for dynamically quantised activations:
 * S = M / max|.| with M = 127, one fp32 division.  *flag is set to 1 (and S = 1) when the
 * maximum is zero or not finite. */
float q8o_scale_from_absmax(float absmax, int *flag)
{
    if (!(absmax > 0.0f) || isinf(absmax)) {
        if (flag) *flag = 1;
        return 1.0f;
    }
    return (float)q8o_M(8) / absmax;
}

/* Eq. 4: running EMA of max|x| over calibration batches.
 * state: ema[0] (fp32), n[0] (batches seen).  Returns S_x = M / ema.
 * decay == 0 keeps no history: the EMA is the maximum of this batch itself, i.e. the scale is exactly
 * the dynamic scale of Sec. 4.1 (no rounding from the update formula). */
float q8o_ema_update(float *ema, int32_t *n, float batch_absmax, float decay, int *flag)
{
    if (*n == 0 || decay == 0.0f) {
        *ema = batch_absmax;
    } else {
        float one_minus_d = 1.0f - decay;
        float diff = batch_absmax - *ema;
        float step = one_minus_d * diff;
        *ema = *ema + step;
    }
    *n += 1;
    return q8o_scale_from_absmax(*ema, flag);
}

/* Eq. 4 on one calibration batch x of `numel` values.  An empty batch carries no observation of max|x|:
 * the state is left as it is and the current scale is returned (1 before any batch has been seen). */
float q8o_calibrate_batch(float *ema, int32_t *n, const float *x, int64_t numel, float decay, int *flag)
{
    if (numel <= 0) return *n == 0 ? 1.0f : q8o_scale_from_absmax(*ema, flag);
    return q8o_ema_update(ema, n, q8o_absmax(x, numel), decay, flag);
}

/* Eq. 1 with Eq. 2 at b = 8: Quantize(x | S, M) = Clamp(nint(x*S), -M, M). */
int8_t q8o_quantize_one(float x, float S)
{
    float p = x * S;                 /* one fp32 multiply (no contraction) */
    if (isnan(p)) return 0;
    float r = rintf(p);              /* nearest integer, halves to even */
    float M = (float)q8o_M(8);
    r = fminf(fmaxf(r, -M), M);      /* Clamp(x,a,b) = min(max(x,a),b) */
    return (int8_t)r;
}

void q8o_quantize(const float *x, int64_t n, float S, int8_t *xq)
{
    for (int64_t i = 0; i < n; ++i) xq[i] = q8o_quantize_one(x[i], S);
}

/* Eq. 3 then Eq. 1 on a weight tensor: returns S_w and fills wq. */
float q8o_quantize_weight(const float *w, int64_t n, int8_t *wq, int *flag)
{
    float S = q8o_scale_from_absmax(q8o_absmax(w, n), flag);
    q8o_quantize(w, n, S, wq);
    return S;
}

/* Sec. 3, inference-mode FC: the GEMM between Int8 inputs, acc[m][n] = sum_k xq[m][k]*wq[n][k].
 * X_q is [M,K] row-major, W_q is [N,K] row-major (Y = X W^T).  Summed in int64 so that an
 * overflow of the Int32 accumulator is detected instead of wrapped: returns the number of
 * entries that do not fit int32 (0 for every K <= 133144). */
int64_t q8o_gemm_s8(const int8_t *xq, const int8_t *wq, int64_t M, int64_t N, int64_t K, int32_t *acc)
{
    int64_t bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k)
                s += (int64_t)xq[m * K + k] * (int64_t)wq[n * K + k];
            if (s > INT32_MAX || s < INT32_MIN) bad += 1;
            acc[m * N + n] = (int32_t)s;
        }
    }
    return bad;
}

/* Sec. 3: the bias is quantised to Int32 with the weights' and activations' scaling factors:
 * b_q = Clamp(nint(b * S_out), -M(32), M(32)), S_out = fl32(S_x * S_w). */
void q8o_quantize_bias(const float *b, int64_t N, float S_x, float S_w, int32_t *bq)
{
    float S_out = S_x * S_w;
    double M32 = (double)q8o_M(32);
    for (int64_t n = 0; n < N; ++n) {
        float p = b[n] * S_out;
        if (isnan(p)) { bq[n] = 0; continue; }
        double r = (double)rintf(p);
        if (r > M32) r = M32;
        if (r < -M32) r = -M32;
        bq[n] = (int32_t)r;
    }
}

/* Sec. 3, inference mode, the Int32 bias add: acc[m][n] += b_q[n] in Int32.  Returns how many sums left
 * the int32 range (they are wrapped to two's complement, as 32-bit hardware would). */
int64_t q8o_add_bias(int32_t *acc, const int32_t *bq, int64_t M, int64_t N)
{
    int64_t bad = 0;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = (int64_t)acc[m * N + n] + (int64_t)bq[n];
            if (s > INT32_MAX || s < INT32_MIN) bad += 1;
            acc[m * N + n] = (int32_t)(uint32_t)(uint64_t)s;
        }
    return bad;
}

/* Inverse of Eq. 1 applied to the product scale: y = acc / (S_x * S_w), in fp64. */
void q8o_dequantize(const int32_t *acc, int64_t count, float S_x, float S_w, double *y)
{
    double denom = (double)S_x * (double)S_w;
    for (int64_t i = 0; i < count; ++i) y[i] = (double)acc[i] / denom;
}

/* GELU, kept in floating point (Sec. 3): y * Phi(y) with the exact erf form, in fp64. */
void q8o_gelu(double *y, int64_t count)
{
    const double inv_sqrt2 = 0.70710678118654752440;
    for (int64_t i = 0; i < count; ++i) y[i] = 0.5 * y[i] * (1.0 + erf(y[i] * inv_sqrt2));
}

/* The whole inference-mode quantised FC layer, step by step.
 *   X [M,K] fp32, Wq [N,K] int8 with its S_w, bias [N] fp32 or NULL, act 0 none / 1 GELU.
 *   S_x_in > 0: static scale (Eq. 4 result);  S_x_in <= 0: dynamic, S_x = M / max|X| (Sec. 4.1).
 * Outputs (caller-allocated): xq [M,K] int8, acc [M,N] int32 (bias included), y [M,N] fp64,
 * *S_x_used.  Return: bit 0 scale flag, bit 1 accumulator overflow. */
int q8o_linear(const float *X, const int8_t *Wq, float S_w, float S_x_in, const float *bias, int act,
               int64_t M, int64_t N, int64_t K, int8_t *xq, int32_t *acc, double *y, float *S_x_used)
{
    int flag = 0, ret = 0;
    float S_x = S_x_in;
    if (!(S_x_in > 0.0f)) S_x = q8o_scale_from_absmax(q8o_absmax(X, M * K), &flag);
    *S_x_used = S_x;
    q8o_quantize(X, M * K, S_x, xq);
    int64_t bad = q8o_gemm_s8(xq, Wq, M, N, K, acc);
    if (bias) {
        int32_t *bq = (int32_t *)malloc((size_t)N * sizeof(int32_t));
        if (!bq) return -1;
        q8o_quantize_bias(bias, N, S_x, S_w, bq);
        bad += q8o_add_bias(acc, bq, M, N);
        free(bq);
    }
    q8o_dequantize(acc, M * N, S_x, S_w, y);
    if (act == 1) q8o_gelu(y, M * N);
    if (flag) ret |= 1;
    if (bad) ret |= 2;
    return ret;
}

/* One output entry of the layer, for spot checks at sizes where the full triple loop is too
 * slow: returns acc+b_q for (m, n) given already-quantised rows. */
int32_t q8o_linear_entry(const int8_t *xq_row, const int8_t *wq_row, int64_t K, int32_t bq)
{
    int64_t s = 0;
    for (int64_t k = 0; k < K; ++k) s += (int64_t)xq_row[k] * (int64_t)wq_row[k];
    s += bq;
    return (int32_t)(uint32_t)(uint64_t)s;
}

/* Sec. 3, inference-mode Embedding: the layer returns the Int8 rows of its table; the fp
 * consumer sees them dequantised, out[t][h] = Eq[ids[t]][h] / S_e (fp64).  rows_q receives
 * the raw Int8 rows.  Returns the number of ids outside [0, V) (those rows are left zero). */
int64_t q8o_embedding(const int32_t *ids, int64_t T, const int8_t *Eq, float S_e, int64_t V, int64_t H,
                      int8_t *rows_q, double *out)
{
    int64_t bad = 0;
    for (int64_t t = 0; t < T; ++t) {
        int64_t id = ids[t];
        if (id < 0 || id >= V) {
            bad += 1;
            for (int64_t h = 0; h < H; ++h) { rows_q[t * H + h] = 0; out[t * H + h] = 0.0; }
            continue;
        }
        for (int64_t h = 0; h < H; ++h) {
            int8_t q = Eq[id * H + h];
            rows_q[t * H + h] = q;
            out[t * H + h] = (double)q / (double)S_e;
        }
    }
    return bad;
}

/* ---- FP32-kept encoder operations (Sec. 3: Softmax and Layer Normalization stay in floating point;
 * the encoder is the BERT of Devlin et al.).  Evaluated in fp64, straight from the definitions. ---- */

/* out[r][:] = LayerNorm(x[r][:] + r1[r][:] + r2[r][:]) * gamma + beta; r1, r2, gamma, beta may be NULL.
 * Mean and (biased) variance over the H features of a row, eps inside the square root. */
void q8o_add_layernorm(const float *x, const float *r1, const float *r2, const float *gamma, const float *beta,
                       double eps, int64_t rows, int64_t H, double *out)
{
    for (int64_t r = 0; r < rows; ++r) {
        double mean = 0.0, var = 0.0;
        for (int64_t h = 0; h < H; ++h) {
            double v = (double)x[r * H + h];
            if (r1) v += (double)r1[r * H + h];
            if (r2) v += (double)r2[r * H + h];
            out[r * H + h] = v;
            mean += v;
        }
        mean /= (double)H;
        for (int64_t h = 0; h < H; ++h) {
            double d = out[r * H + h] - mean;
            var += d * d;
        }
        var /= (double)H;
        double rstd = 1.0 / sqrt(var + eps);
        for (int64_t h = 0; h < H; ++h) {
            double g = gamma ? (double)gamma[h] : 1.0, b = beta ? (double)beta[h] : 0.0;
            out[r * H + h] = (out[r * H + h] - mean) * rstd * g + b;
        }
    }
}

/* Multi-head self-attention without mask: qkv [B*S][3*heads*d] = [q | k | v] per token,
 * ctx[b][i][h] = sum_j softmax_j(q_i . k_j / sqrt(d)) v_j. */
void q8o_attention(const float *qkv, int64_t B, int64_t S, int64_t heads, int64_t d, double *ctx)
{
    int64_t H = heads * d, P = 3 * H;
    double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t hd = 0; hd < heads; ++hd) {
            double *score = (double *)malloc((size_t)S * sizeof(double));
            for (int64_t i = 0; i < S; ++i) {
                const float *q = qkv + (b * S + i) * P + hd * d;
                double mx = -INFINITY, sum = 0.0;
                for (int64_t j = 0; j < S; ++j) {
                    const float *k = qkv + (b * S + j) * P + H + hd * d;
                    double s = 0.0;
                    for (int64_t t = 0; t < d; ++t) s += (double)q[t] * (double)k[t];
                    score[j] = s * scale;
                    if (score[j] > mx) mx = score[j];
                }
                for (int64_t j = 0; j < S; ++j) {
                    score[j] = exp(score[j] - mx);
                    sum += score[j];
                }
                for (int64_t t = 0; t < d; ++t) {
                    double acc = 0.0;
                    for (int64_t j = 0; j < S; ++j) acc += score[j] * (double)qkv[(b * S + j) * P + 2 * H + hd * d + t];
                    ctx[(b * S + i) * H + hd * d + t] = acc / sum;
                }
            }
            free(score);
        }
    }
}

/* ---- Training-mode pieces (Sec. 2.2, Sec. 3 "During training ..."): fake quantisation simulates the rounding
 * in floating point, x_hat = Quantize(x | S, M) / S, and the straight-through estimator (Eq. 5) passes the
 * gradient through unchanged. ---- */
void q8o_fake_quantize(const float *x, int64_t n, float S, double *xhat)
{
    for (int64_t i = 0; i < n; ++i) xhat[i] = (double)q8o_quantize_one(x[i], S) / (double)S;
}

/* Eq. 5: d x_hat / d x = 1 for every element. */
void q8o_ste_backward(const float *grad_out, int64_t n, double *grad_in)
{
    for (int64_t i = 0; i < n; ++i) grad_in[i] = (double)grad_out[i];
}
