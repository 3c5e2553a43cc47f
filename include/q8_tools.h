/*
 * q8_tools.h -- tuning hooks, measurement aids and a self-test entry of libq8.
 *
 * None of these has a counterpart in the paper and none is needed to run the quantised layers of q8.h:
 * they exist for benchmarks, profiling and tests.  They live in the same shared library.  The tuning hooks
 * set process-global switches and are not thread-safe; results of the q8.h calls never depend on them.
 */
#ifndef Q8_TOOLS_H_
#define Q8_TOOLS_H_

#include "q8.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Tuning / test hook: force the tile shape of the tcgen05 GEMM for later calls in this process.
 * (block_n, ctas) = (0, 0) restores the automatic choice; otherwise ctas = 1 with block_n in
 * {32, 64, 128, 256} (one SM per 128 x block_n tile) or ctas = 2 with block_n = 256 (a pair of
 * SMs per 256 x 256 tile).  Results do not depend on the choice.  Not thread-safe. */
q8_status q8_tune_gemm_tile(int block_n, int ctas);

/* Tuning / test hook: epilogue warps per CTA of the cta_group::2 kernel for later calls in this process:
 * 8 (each warp walks four 32-column blocks per tile), 16 (two blocks per warp) or 0 = automatic.  Other values are Q8_ERR_ARG.  Results do not depend on it. */
q8_status q8_tune_gemm_epilogue_warps(int warps);

/* Tuning / test hook for the schedule of the cta_group::2 kernel.  When the number of 256 x 256 tiles
 * is not a multiple of the number of SM pairs, the tiles of the last, partial round are cut into 2 or 4
 * narrower tiles (256 x 128 or 256 x 64) if these still fit in one round, which shortens that round.
 * enable = 0 switches this off for later calls in this process, non-zero (the default) on.  Results do
 * not depend on it.  Not thread-safe.  (An implementation detail with no counterpart in the paper.) */
void q8_tune_gemm_tail_split(int enable);

/* Tuning / test hook for the way the tcgen05 GEMM writes a plain fp32 output (no Int8 copy asked for).
 * mode 1: each epilogue warp reads its accumulator block in the 16 x 256 bit fragment layout and stores it
 * straight from registers, every 32-byte sector written whole by four neighbouring lanes (CTA-pair kernel only, and
 * only when neither an Int8 copy nor the debug accumulator is asked for); mode 0: the block
 * is staged in shared memory and leaves as a TMA store; mode < 0 (the default): automatic, unstaged only for the
 * CTA-pair kernel with the 8-warp epilogue (K > 2048), where it measured 2 % faster.  Results do not depend on
 * it.  Not thread-safe. */
void q8_tune_gemm_direct_store(int mode);

/* Into how many narrower tiles each tile of the last round was cut by the most recent tcgen05 GEMM launch
 * of this host thread: 1 (not cut), 2 or 4. */
int q8_last_launch_tail_split(void);

/* How the most recent tcgen05 GEMM launch of this host thread wrote its fp32 output: 0 every lane stored its own
 * row (Y not aligned for a TMA store, or no fp32 output), 1 staged in shared memory and stored by TMA, 2 stored
 * straight from the accumulator fragments (see q8_tune_gemm_direct_store). */
int q8_last_launch_store_mode(void);

/* Tuning / test hook: q8_attention / q8_attention_quant use the tensor-core kernel when the shape allows it
 * (non-zero, the default) or always the CUDA-core fp32 kernel (0), for later calls in this process. */
void q8_tune_attention(int use_tensor_cores);

/* Measurement aid, no counterpart in the paper: the issue-bound Int8 rate of the tensor cores of the current
 * device, i.e. the ceiling of the GEMM's tensor pipe when operands cost nothing.  Every SM (ctas = 1) or SM
 * pair (ctas = 2, cta_group::2) issues the GEMM kernel's own tcgen05.mma kind::i8 shape (M = 128 * ctas,
 * N = 256, K = 32) back to back on operand tiles that stay in shared memory (pseudo-random bytes; no TMA, no
 * stores) for about `seconds` (0 < seconds <= 5; a short calibration launch sizes the timed launch).
 * Host outputs: *tops = 2 M N K * instructions / time in 1e12 op/s (required), *elapsed_ms and *sms_used
 * (either may be NULL).  `dev_status` (device int32, may be NULL) receives Q8_ERR_TIMEOUT bits should a wait
 * inside the kernel give up.  Synchronises `stream`.  Returns Q8_ERR_ARG on bad arguments, Q8_ERR_CUDA when a
 * runtime call fails. */
q8_status q8_measure_int8_mma_peak(int ctas, double seconds, double *tops, double *elapsed_ms, int *sms_used,
                                   void *dev_status, void *stream);

/* Measurement aid, no counterpart in the paper: the one-directional HBM rates of the current device.  A copy
 * moves one byte in per byte out; the FC layers write 4 M N bytes of fp32 against M K + N K bytes of Int8
 * operands, so what bounds their output-heavy shapes is the store-only rate, which is well below the copy rate.
 * `buf` (device, 16-byte aligned, caller-owned, at least `bytes` long; make it several times the L2 size) is
 * overwritten with a pattern `repeats` times (store != 0) or read `repeats` times (store == 0) by a plain
 * grid-stride kernel of 16-byte accesses after one untimed pass.  Host outputs: *gbs = bytes * repeats / time in
 * 1e9 B/s (required), *elapsed_ms (may be NULL).  Synchronises `stream`.  Allocates no device memory.
 * Returns Q8_ERR_NULL / Q8_ERR_ALIGN / Q8_ERR_ARG (bytes < 16, repeats outside 1..1000) / Q8_ERR_CUDA. */
q8_status q8_measure_hbm_peak(void *buf, size_t bytes, int store, int repeats, double *gbs, double *elapsed_ms,
                              void *stream);

/* Measurement aid, no counterpart in the paper: the rate (GB/s, over all SMs) at which TMA pulls L2-resident
 * operand boxes (128 rows x 128 bytes, the GEMM's operand box) into shared memory, with nothing else running:
 * the ceiling of the GEMM's main loop when no operand byte is shared between SMs.  buf (device, 16-byte aligned)
 * is read as a row-major Int8 matrix [rows, K] (rows % 128 == 0, K % 128 == 0; keep rows * K well below the L2
 * size so that the timed launch reads from L2); every SM loads boxes_per_sm boxes through a ring of 12 stages.
 * sms_used = 0 runs one CTA on every SM, a smaller positive number that many CTAs (to tell a per-SM limit from
 * a limit of the L2 side).  producers = 1, 2, 3 or 4 warps issue the loads, each into its own share of the ring
 * (one warp alone is bound by its own issue loop, about a box per 285 cycles).
 * One untimed launch warms L2, the next is timed with CUDA events.  *gbs and *elapsed_ms (may be NULL) are host
 * outputs.  Returns Q8_ERR_TIMEOUT if a bounded wait inside the kernel ran out.  Synchronises the stream. */
q8_status q8_measure_l2_operand_peak(const void *buf, int64_t rows, int64_t K, int boxes_per_sm, int sms_used,
                                     int producers, double *gbs, double *elapsed_ms, void *stream);

/* Self-test of the bounded device-side wait every tensor-core kernel of the library is built on.  Launches one
 * small CTA that initialises an mbarrier nobody ever arrives on and waits on it with the library's own bounded
 * wait, limited to `limit_ns` nanoseconds (1000 <= limit_ns <= 100 000 000).  The wait must give up: the kernel
 * then ORs (1 << Q8_ERR_TIMEOUT) into *dev_status (device int32, required), writes how the wait ended into
 * dev_report (device int32[2], optional: [0] = 1 if the wait reported failure, [1] = the CTA's abort flag) and
 * returns normally, leaving the context usable.  Nothing spins without limit and nothing traps.  Asynchronous on
 * `stream`; read the result with q8_poll_status. */
q8_status q8_selftest_wait_timeout(uint64_t limit_ns, int32_t *dev_status, int32_t *dev_report, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* Q8_TOOLS_H_ */
