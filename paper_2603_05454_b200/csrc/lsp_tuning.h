/*
 * lsp_tuning.h -- internal knobs of the B200 LSP decode library, for the micro-benchmarks and the kernel tests.
 *
 * Not part of the public contract (include/lsp.h): the keys name tile shapes, grids and benchmark aids of the current
 * kernels and change with them.  None of them changes what the library computes, except keys 3-5, which change how
 * lsp_op_linear behaves as a timing harness.
 */
#ifndef LSP_TUNING_H_
#define LSP_TUNING_H_

#include "../../include/lsp.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Benchmark aids:
 *   3  lsp_op_linear returns without synchronising or checking the device status (1) or not (0)
 *   4  lsp_op_linear enqueues the operation this many times
 *   5  repetition r reads its weights at W + (r mod value) * N * K elements, so a buffer of several weight copies keeps
 *      the L2 cold
 * tcgen05 GEMM (the persistent kernel k_gemm_stream):
 *   10 CTAs a launch whose tiles are split is dealt to (0 = by the tile count)          11 maximum pipeline stages
 *   17 grid of the persistent kernel (0 by row count, 1 one CTA per SM with even shares, 2 a multiple of the tile count)
 *   18 row count up to which mode 0 takes even shares
 *   19 129..256 rows: 1 = two row tiles per CTA (default), 2 = two row groups
 *   20 its tile width for those (0 = automatic, 128, 256)
 *   21 64-element K atoms per pipeline stage (0 = automatic, 1, 2)   22 fewest two-atom stages the automatic choice accepts
 *   23 its tile width for up to 128 rows (0 = automatic, 128, 256)
 *   24 row tiles per CTA above 256 rows (1, 2, 3 = automatic, default)
 *   25 launch the step's kernels with programmatic dependent launch (1, default) or plainly (0)
 *   26 MMA-issuing warps of the persistent kernel with one row tile per CTA (1, default, or 2)
 *   27 the persistent kernel caps its shared memory at half an SM when three stages still fit (1, default)
 *   29 the K slices of a split tile run as one thread block cluster, reduced through distributed shared memory (1,
 *      default), or through global scratch by the last CTA to arrive (0)
 *   32 tile width of the dual (SwiGLU) GEMM: 0 = automatic (default), 192 or 256
 *   33 a cluster of 2 exchanges half tiles (1, default) or publishes whole partial tiles like larger clusters (0)
 * tcgen05 attention:
 *   28 fewest (query row x group head) rows of a (sequence, KV head) for which the tcgen05 kernel is used (default 0)
 *   30 it splits a row tile's keys over a thread block cluster when there are few CTAs (1, default)
 *   39 with 129..192 rows on two row tiles and unsplit tiles, the second row tile's MMAs span 64 rows (1, default)
 *   36, 37 fewest and most activation rows of a GEMM that takes the operand-swapped kernel (defaults 129 and 256;
 *      37 = 0: never)        38 take it whenever it can run (1), not only where it was measured to pay (0, default)
 * decode loop:
 *   31 with device-resident block lengths (lsp_set_option key 4), lsp_generate reads every step before sizing the next
 *      once at most this many masked positions per sequence remain (default 8)
 * Unknown key: LSP_ERR_ARG. */
int lsp_debug_set(lsp_ctx* ctx, int key, int value);

/* Exercises the bounded-wait recovery path without touching any data: launches one thread that waits, for limit_us
 * microseconds, on a barrier nothing arrives at, and then records the expiry in the context's status word the way the
 * GEMM and attention kernels do.  Returns what a step would return in that situation: LSP_ERR_DEVICE_TIMEOUT (site 99
 * in lsp_last_error), with the status word and the split-K counters cleared again, so that the next call runs normally. */
int lsp_debug_wait_selftest(lsp_ctx* ctx, int limit_us);

#ifdef __cplusplus
}
#endif
#endif /* LSP_TUNING_H_ */
