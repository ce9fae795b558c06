/*
 * mlmc_instr.h: measurement and debugging aids of the MLMC library.  Nothing here is part of the
 * method (the paper has no counterpart): launch accounting, per-kernel CUDA-event timing, the
 * uniforms of the level draw for known-answer checks, and how much of a row the last Top-k emission
 * read.  The calls that copy to the host synchronise the stream they are given.
 */
#ifndef MLMC_INSTR_H
#define MLMC_INSTR_H

#include "mlmc.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Number of kernels this ctx has launched so far (host counter; for launch accounting). */
int64_t mlmc_launch_count(const mlmc_ctx* ctx);

/* Per-kernel timing for roofline measurements (instrumentation of this library; not part of the
 * method).  With timing on, every kernel launch is bracketed by a CUDA event pair on its stream (at
 * most 2048 launches between two reads; later ones are not recorded).  mlmc_timing_read synchronises
 * `stream`, fills total_ms[id] and launches[id] for id < mlmc_kernel_count() (host arrays) with the
 * launches recorded since the previous read, and restarts the record. */
int mlmc_kernel_count(void);
const char* mlmc_kernel_name(int id);
int mlmc_timing_enable(mlmc_ctx* ctx, int on);
int mlmc_timing_read(mlmc_ctx* ctx, double* total_ms, int64_t* launches, void* stream);

/* The uniforms of the level draw for workers 0..M-1 at (seed, step), computed on the device and
 * copied to u_host[M].  Synchronous; for checking the counter generator against known answers. */
int mlmc_read_u(mlmc_ctx* ctx, uint64_t seed, uint64_t step, int M, double* u_host, void* stream);

/* How much of every row the last mlmc_compress_topk / mlmc_compress_stopk on this context read when it emitted the
 * bands (the band of ranks (k_{l-1}, k_l] of Sec. 3.2): the emission reads only the batches of 512 32-bit words
 * (512 fp32 or 1024 bf16 entries; eight batches make a tile) whose largest magnitude reaches the band's lower
 * threshold, twice each.
 *   listed_host  host uint32 [M]: batches of worker m that were read.
 *   tiles_host   host int64: batches in one row (the ragged last tile counted whole).
 * Synchronous (copies from the device and waits for the stream); a measurement aid, not part of the method. */
int mlmc_read_listed_tiles(mlmc_ctx* ctx, int M, uint32_t* listed_host, int64_t* tiles_host, void* stream);

/* Fixed-p Top-k on fp32 reuses, per worker and level boundary, the leading-digit bin in which the threshold was
 * found by the last call on the same problem (same d, M, schedule, dtype) as a bracket: the first sweep collects the
 * keys of that bin and its two neighbours, and when the new threshold bins fall inside, no second pass over the
 * gradient is made for the candidates (Sec. 3, remark after Alg. 2: the residual without computing each term).
 *   stats_host  host uint64[3], cumulative since mlmc_create: workers whose two brackets both held / workers with a
 *               bracket that missed (the candidate pass ran) / workers without a stored bin yet.
 * Synchronous; a measurement aid. */
int mlmc_read_bracket_stats(mlmc_ctx* ctx, uint64_t* stats_host, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MLMC_INSTR_H */
