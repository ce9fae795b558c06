/*
 * mlmc.h: C ABI of the MLMC gradient-compression hot path (CUDA, sm_100a).
 *
 * The library turns a biased multilevel compressor C^l (Def. 3.1) into the unbiased MLMC estimate
 *     g~ = g^0 + (1/p^l)(C^l(g) - C^{l-1}(g)),   g^0 = 0,   l ~ p            (Eq. 5; Alg. 2 / Alg. 3)
 * for each of M workers, emits each worker's message, and averages the M messages on the server
 * side (Alg. 2, "Server aggregates").  Two compressor families are covered: Top-k with a level
 * schedule k_0 <= ... <= k_{L-1} = d (Sec. 3.2) and fixed-point bit truncation with a bit schedule
 * b_0 < ... < b_{L-1} <= 23 (Sec. 3.1).  Probabilities are either given (Alg. 2) or adaptive,
 * p^l proportional to ||C^l(g) - C^{l-1}(g)||_2 per worker per step (Lemma 3.4, Alg. 3).
 *
 * Conventions
 *  - Levels are indexed l = 0..L-1 here; this is the paper's l = 1..L.  k_{-1} = 0, b_{-1} = 0.
 *  - Pointers are DEVICE pointers unless marked "host".  The caller owns every buffer; the library
 *    only owns the scratch workspace inside mlmc_ctx.
 *  - All work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL = default
 *    stream).  Nothing synchronises except mlmc_create, mlmc_destroy and mlmc_get_status (and the
 *    measurement calls of mlmc_instr.h, which are not part of the method).
 *  - The int return value reports host-side checks made before any launch (arguments, schedule,
 *    probabilities).  Conditions found on the device (message capacity, non-finite input, a bounded
 *    wait that gave up) are written to a sticky status word read by mlmc_get_status; the affected
 *    worker's message then has count = 0 (Top-k) or level = -1.  Nothing traps or spins unbounded.
 *  - g is [M][ld] with row stride ld >= d elements, worker m in row m; g must be 16-byte aligned and,
 *    when M > 1, ld * sizeof(element) must be a multiple of 16.  d < 2^32.  g is never written.
 *  - Total order for Top-k: |g_i| descending, equal magnitudes by ascending index i.
 *  - One uniform per (seed, step, worker) drives the level draw: three chained SplitMix64 output
 *    rounds, u = (h >> 11) * 2^-53; cdf accumulated in ascending l in fp64, the cdf of the last level
 *    with p > 0 set to 1, l* = min{ l : u < cdf_l }.
 *  - One mlmc_ctx serves one stream at a time.  Contexts share nothing: calls on different contexts may run
 *    side by side on different streams.
 */
#ifndef MLMC_H
#define MLMC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mlmc_ctx mlmc_ctx;

typedef enum { MLMC_F32 = 0, MLMC_BF16 = 1 } mlmc_dtype;
typedef enum { MLMC_TOPK = 0, MLMC_BITWISE = 1, MLMC_RTN = 2 } mlmc_kind;

typedef enum {
    MLMC_OK = 0,
    MLMC_ERR_ARG = -1,       /* null pointer, size out of range, misaligned g, limits of the ctx exceeded */
    MLMC_ERR_SCHEDULE = -2,  /* k not nondecreasing or k_{L-1} != d;  b not increasing or b_{L-1} > 23 */
    MLMC_ERR_PROB = -3,      /* some p_l <= 0 or sum p != 1 (Lemma 3.2 needs non-zero probabilities) */
    MLMC_ERR_CAPACITY = -4,  /* device: a Top-k message does not fit out->capacity / planes exceed w_max */
    MLMC_ERR_NONFINITE = -5, /* device: NaN or Inf in g */
    MLMC_ERR_TIMEOUT = -6,   /* reserved (no kernel of this version waits for another thread block) */
    MLMC_ERR_CUDA = -7,      /* a CUDA runtime call failed */
    MLMC_ERR_NOMEM = -8,     /* workspace allocation failed */
    MLMC_ERR_INTERNAL = -9   /* device: a self-check failed (emitted count differs from k_l - k_{l-1}) */
} mlmc_status;

#define MLMC_MAX_LEVELS 32

/* Top-k message batch (Sec. 3.2: the residual C^l - C^{l-1} is the band of ranks (k_{l-1}, k_l]).
 * Structure of arrays in device memory.  Worker m owns idx[m*capacity ..] and val[m*capacity ..]. */
typedef struct {
    uint32_t* idx;     /* [M][capacity] coordinates of the band, ascending                         */
    float*    val;     /* [M][capacity] g_i / p_l                                                  */
    int64_t*  count;   /* [M] entries written = k_l - k_{l-1}; 0 if the worker hit a device error  */
    int32_t*  level;   /* [M] sampled level l*, or -1 on a device error                            */
    double*   p_sel;   /* [M] probability of the sampled level                                     */
    int64_t   capacity;/* entries per worker; max_l (k_l - k_{l-1}) always suffices                */
} mlmc_topk_msgs;

/* Bit-plane message batch (Sec. 3.1: the residual of the fixed-point code is the level's bit
 * field plus a sign bit per entry; with the unit schedule b_l = l+1 that is 2 bits per entry).
 * Worker m owns planes[m * (1+w_max) * words ..], words = ceil(d/32).  Plane 0 holds the raw sign
 * bits, plane j = 1..w_l holds bit (w_l - j) of the field (most significant first); bit t of word w
 * is coordinate 32 w + t; bits past d are 0; planes past 1 + w_l are not written. */
typedef struct {
    uint32_t* planes;  /* [M][1 + w_max][ceil(d/32)]                                               */
    float*    gmax;    /* [M] max_i |g_i|, the normaliser sent with the message                    */
    int32_t*  level;   /* [M] sampled level, or -1 on a device error                               */
    double*   p_sel;   /* [M]                                                                      */
    int32_t   w_max;   /* magnitude planes allocated per worker; need >= max_l (b_l - b_{l-1})     */
} mlmc_bit_msgs;

/* Allocates the scratch workspace for problems up to (d_max, M_max, L_max) on `device`.
 * Synchronous.  L_max <= MLMC_MAX_LEVELS, M_max <= 1024.  Returns MLMC_ERR_NOMEM / MLMC_ERR_CUDA on failure. */
int mlmc_create(mlmc_ctx** ctx, int device, int64_t d_max, int M_max, int L_max);
int mlmc_destroy(mlmc_ctx* ctx);

/* Synchronises `stream`, returns the sticky device status (first error since the last call) and clears it. */
int mlmc_get_status(mlmc_ctx* ctx, void* stream);

/* Level probabilities and residual norms (Lemma 3.4; Alg. 3 "Compute p^l = Delta^l / sum Delta").
 *   kind   MLMC_TOPK: sched = host int64 k[L];  MLMC_BITWISE: sched = host int64 b[L];
 *          MLMC_RTN: sched = host int64 r[L-1] (the widths of mlmc_compress_rtn; level L-1 is the identity).
 *   p_host NULL: adaptive, p_out[m][l] = Delta_l / sum Delta (all weight on level 0 if every Delta is 0).
 *          else: host double[L], all > 0, sum 1 within 1e-9; p_out[m][l] = p_host[l] / sum.
 *   p_out     device double [M][L].
 *   delta_out device double [M][L] or NULL: Delta_l = ||C^l(g) - C^{l-1}(g)||_2 (always computed from g). */
int mlmc_level_probs(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, int kind,
                     const int64_t* sched, int L, const double* p_host, double* p_out, double* delta_out,
                     void* stream);

/* MLMC-Top-k message of every worker (Alg. 2 / Alg. 3, the lines from "Sample l" to "Send").
 *   k host int64[L], nondecreasing, k[L-1] = d (Def. 3.1: the top level is the identity).
 *   p host double[L] or NULL for adaptive.  (seed, step, row index m) select the uniform of worker m.
 * Device errors: capacity < band size -> MLMC_ERR_CAPACITY; NaN/Inf -> MLMC_ERR_NONFINITE. */
int mlmc_compress_topk(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld,
                       const int64_t* k, int L, const double* p, uint64_t seed, uint64_t step,
                       const mlmc_topk_msgs* out, void* stream);

/* MLMC fixed-point bit-wise message of every worker (Sec. 3.1).
 *   b host int32[L], strictly increasing, b[L-1] = B <= 23.
 *   Code: e_i = fl32(|g_i| / gmax) (IEEE division), q_i = min(floor(e_i 2^B), 2^B - 1);
 *   level l keeps the top b_l bits of q; field f_l = (q >> (B - b_l)) & (2^{w_l} - 1), w_l = b_l - b_{l-1};
 *   residual entry = sign_i f_l 2^{-b_l} gmax;  adaptive Delta_l = gmax 2^{-b_l} sqrt(sum_i f_l^2). */
int mlmc_compress_bitwise(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld,
                          const int32_t* b, int L, const double* p, uint64_t seed, uint64_t step,
                          const mlmc_bit_msgs* out, void* stream);

/* Server average (Alg. 2 / Alg. 3 "Server aggregates: (1/M) sum_i g~_i") into dense out[d] (fp32,
 * every element written exactly once).  kind selects the message struct msgs points to (host
 * struct holding device pointers).  b host int32[L] for MLMC_BITWISE, ignored for MLMC_TOPK.
 * Terms are added in worker order 0..M-1 in fp32, so the result is reproducible run to run.
 * Workers whose level is -1 contribute nothing. */
int mlmc_aggregate(mlmc_ctx* ctx, int kind, const void* msgs, const int32_t* b, int L, int M, int64_t d,
                   float* out, void* stream);

/* ---- Further multilevel compressors of the paper, same estimator (Eq. 5), same draw, same server average. ---- */

/* s-Top-k (Sec. 2.2 "s-segmented Top-k"; App. D: the segments are those of the sorted vector): level l keeps
 * the l + 1 segments of length s of largest norm, i.e. Top-(s (l + 1)); L = ceil(d / s) levels, at most
 * min(2^20, d_max of the context); the residual of level l is the l-th segment (Sec. 3.2), at most s entries, so
 * capacity >= min(s, d) suffices.
 *   p  host double[L], all > 0, sum 1 (Alg. 2), or NULL for adaptive p (Lemma 3.4: p^l proportional to the norm of
 *      segment l).
 * Up to MLMC_MAX_LEVELS segments run through mlmc_compress_topk with the schedule k_l = min(d, s (l + 1)).  With more
 * segments and a given p the level is drawn before the data is read and only the two thresholds of its segment are
 * selected.  With more segments and adaptive p every segment norm is needed: each row's magnitude keys are sorted
 * (radix sort, about ten sweeps of the row), as many rows together as fit in 1 GiB of scratch memory (about
 * 8 d_max + 8 min(2^20, d_max) bytes per row; at least one row), which the first such call on a context takes with
 * one cudaMalloc (MLMC_ERR_NOMEM if it fails; freed by mlmc_destroy).
 * Returns MLMC_ERR_ARG when L exceeds the limit. */
int mlmc_compress_stopk(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, int64_t s,
                        const double* p, uint64_t seed, uint64_t step, const mlmc_topk_msgs* out, void* stream);

/* Floating-point bit-wise message batch (Sec. 2.2 "Floating-point compressors", App. B): sign and exponent of
 * every entry are always sent, level l adds the mantissa digits mb_{l-1}+1 .. mb_l (one digit per entry for the
 * unit schedule: the paper's 1 + exponent + 1 bits per entry).
 *   expo    [M][32 ceil(d/32)] bytes: biased exponent field of entry i of worker m at expo[m * 32 * words + i].
 *   planes  [M][1 + w_max][ceil(d/32)]: plane 0 = raw sign bits, plane j = bit (w_l - j) of the mantissa field. */
typedef struct {
    uint8_t*  expo;
    uint32_t* planes;
    int32_t*  level;   /* [M] sampled level, or -1 on a device error (NaN / Inf in g)                 */
    double*   p_sel;   /* [M]                                                                         */
    int32_t   w_max;   /* magnitude planes allocated per worker; need >= max_l (mb_l - mb_{l-1})      */
} mlmc_float_msgs;

/* MLMC with the floating-point compressor (App. B).  C^l(e) keeps sign, exponent and the first mb_l mantissa
 * digits of every entry; mb host int32[L], strictly increasing, mb[L-1] = 23 for fp32 and 7 for bf16 input (the top
 * level is the identity, Def. 3.1).  The estimate is g^0 + (1/p^l)(C^l - C^{l-1}) with the always-sent part
 * g^0 = sign 2^(E - bias) (an entry with exponent field 0 has g^0 = 0 and the scale of exponent field 1).
 *   p  host double[L] or NULL: NULL takes App. B's optimal fixed probabilities, p^l proportional to 2^-l for the
 *      unit schedule, in general to the largest residual of the level, 2^-mb_{l-1} - 2^-mb_l.
 * One sweep over g; the level draw does not depend on the data.  expo and planes must be 16-byte aligned. */
int mlmc_compress_floatbits(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld,
                            const int32_t* mb, int L, const double* p, uint64_t seed, uint64_t step,
                            const mlmc_float_msgs* out, void* stream);

/* Server average of floating-point messages into dense out[d] (fp32, worker order 0..M-1). */
int mlmc_aggregate_floatbits(mlmc_ctx* ctx, const mlmc_float_msgs* msgs, const int32_t* mb, int L, int M, int64_t d,
                             float* out, void* stream);

/* MLMC-RTN message batch (Sec. 3.2 end, App. G): the residual of a round-to-nearest level has no sparse or
 * bit-plane structure, so the message is the dense vector (C^l - C^{l-1}) / p^l. */
typedef struct {
    float*   val;      /* [M][ldv] dense residual scaled by 1/p, row stride ldv >= d elements, 16-byte aligned rows */
    float*   c;        /* [M] clipping value c = max_i |g_i|                                                       */
    int32_t* level;    /* [M] sampled level, or -1 on a device error                                               */
    double*  p_sel;    /* [M]                                                                                      */
    int64_t  ldv;
} mlmc_rtn_msgs;

/* MLMC with round-to-nearest levels (App. G): C^l(v) = clip(delta^l round(v / delta^l), -c, c),
 * delta^l = 2c / (2^{r_l} - 1), for bit widths r host int32[L-1], strictly increasing, r <= 16; level L-1 is the
 * identity (Def. 3.1).  The rounding is fixed as: inv = fl32((2^r - 1) / (2c)), delta = fl32(2c / (2^r - 1)),
 * t = fl32(v inv), k = t rounded to nearest (ties to even), C = clip(fl32(k delta), -c, c); residuals, their norms
 * and the scaling by 1/p are fp64, the message value is rounded to fp32 once.
 *   p  host double[L] or NULL for adaptive p (Lemma 3.4, Alg. 3; the paper's MLMC-RTN is adaptive). */
int mlmc_compress_rtn(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* r, int L,
                      const double* p, uint64_t seed, uint64_t step, const mlmc_rtn_msgs* out, void* stream);

/* Server average of dense messages: out[i] = (1/M) sum_m val[m][i], workers with level -1 left out. */
int mlmc_aggregate_rtn(mlmc_ctx* ctx, const mlmc_rtn_msgs* msgs, int M, int64_t d, float* out, void* stream);

/* The Top-k case of mlmc_aggregate for callers that must not allocate device memory.  (The paper
 * has no counterpart: this is a deployment variant of the same averaging step.)
 *
 * mlmc_aggregate keeps a small table of tile offsets in the workspace of an mlmc_ctx, and creating a
 * context calls cudaMalloc.  Code that runs after a framework has claimed the whole GPU for its own
 * memory pool, inside a region where the allocator may not be entered (a real-time loop, a callback
 * from another library, a process whose memory budget is fixed at start-up), cannot do that.  This
 * entry point needs no context: its table lives in a device array compiled into the library, 4 MiB
 * that every GPU which loads the library holds until the process exits.  It calls neither cudaMalloc
 * nor cudaFree nor any routine that allocates.
 *
 *   msgs, out   as for mlmc_aggregate with kind MLMC_TOPK: host struct of device pointers, dense out[d].
 *   Limit       M * (ceil(d / 4096) + 1) <= 2^20; larger problems return MLMC_ERR_ARG and nothing is launched.
 *   Device      the current device of the calling thread; msgs and out must live there.
 *   First call  on each device looks up the device address of the built-in table (a synchronous
 *               runtime query); make that first call before starting any stream capture.  Host threads
 *               may make their first calls on a device concurrently: the looked-up values are published
 *               with release/acquire ordering and looking them up twice is harmless.
 *   Sharing     every call on a device uses the same table.  Each call rewrites all entries it reads,
 *               so nothing carries over between calls, but two calls whose kernels overlap on the GPU
 *               (different streams, or several host threads) race: run them one after the other.
 * The result is identical to mlmc_aggregate's on the same messages. */
int mlmc_aggregate_topk_noalloc(const mlmc_topk_msgs* msgs, int M, int64_t d, float* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MLMC_H */
