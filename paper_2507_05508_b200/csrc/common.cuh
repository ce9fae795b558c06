// Shared declarations of the MLMC CUDA library: workspace layout, device helpers, launcher prototypes.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mlmc.h"
#include "../../include/mlmc_instr.h"

namespace mlmc {

constexpr int kMaxLevels = MLMC_MAX_LEVELS;   // L <= 32, so at most 31 thresholds per worker
constexpr int kMaxQueries = kMaxLevels;
constexpr int kBins1 = 32768;                 // leading digit: key bits 30..16 (fp32) / the whole key (bf16)
constexpr int kBins23 = 256;                  // second and third digits: key bits 15..8 and 7..0
constexpr uint32_t kKeyNone = 0xFFFFFFFFu;    // threshold above every finite key: "nothing is inside"
constexpr uint32_t kNoSlot = 0xFFu;

constexpr int kSweepThreads = 512;            // histogram / masked / norm sweeps
constexpr int kEmitMaxWorkers = 1024;         // M of one call: the emit and averaging kernels keep per-worker offsets in shared memory
constexpr int kEmitRows = 16;                 // 32-bit words per lane that a warp of the emit kernels holds at a time
constexpr int kEmitTile = 4096;               // 32-bit words per emit tile (1 fp32 or 2 bf16 elements each); one warp per tile
constexpr int kEmitTileVecs = kEmitTile / 4;  // 16-byte vectors per tile, for both element types
constexpr int kEmitGroups = kEmitTile / (kEmitRows * 32);  // batches of kEmitRows * 32 words per tile: 8
constexpr int kEmitGroupVecs = kEmitTileVecs / kEmitGroups;  // 16-byte vectors per batch: 128
constexpr int kAggTile = 4096;                // dense output elements per aggregation tile

// Per-worker selection query: the rank-k element of the total order.
struct Query {
    uint32_t k;        // target rank, 1 <= k < d for live queries
    uint32_t prefix;   // key bits fixed so far
    uint32_t rem;      // rank still to descend inside the current prefix set (1-based, from the top)
    uint32_t slot;     // histogram slot of the next digit pass (kNoSlot when resolved or trivial)
    uint32_t T;        // resolved threshold key
    uint32_t c;        // #{ key > T }
    uint32_t n;        // #{ key == T }
    uint32_t r;        // how many key == T elements, in index order, are inside Top-k  (k - c)
    uint32_t trivial;  // 1: k == 0 (nothing inside), 2: k >= d (everything inside), 0: live
    uint32_t pad[3];
};

// Emit parameters of one worker, produced by the draw kernel.
struct EmitParams {
    uint32_t Ta, ra;   // Top-k_{l*-1}: inside iff key > Ta or (key == Ta and tie rank <= ra)
    uint32_t Tb, rb;   // Top-k_{l*}
    double inv_p;      // 1 / p_{l*}
    uint32_t expect;   // k_{l*} - k_{l*-1}
    int32_t enabled;   // 0: worker skipped (device error)
    int32_t level;
    int32_t pad;
};

// Kernel identifiers for launch accounting and per-kernel timing.
enum KernelId {
    K_DRAW_FIXED = 0, K_INIT_QUERIES, K_UNIFORMS, K_HIST1, K_RESOLVE1, K_SUMS_CAND, K_CAND2, K_MASKED2, K_RESOLVE2, K_CAND3,
    K_MASKED3, K_RESOLVE3, K_CAND_SUMS, K_NORM_SWEEP, K_NORM_HIST, K_PROBS_DRAW, K_COPY_PROBS, K_EMIT, K_AGG_OFFSETS, K_AGG_TOPK,
    K_ABSMAX, K_BIT_STATS, K_BIT_DRAW, K_BIT_PACK, K_AGG_BIT, K_TILE_LIST, K_BAND_COUNT, K_BAND_SCAN, K_BIT_PACK_WIDE, K_RESET,
    K_FLOAT_DRAW, K_FLOAT_PACK, K_AGG_FLOAT, K_RTN_STATS, K_RTN_DRAW, K_RTN_EMIT, K_AGG_DENSE, K_STOPK_DRAW, K_STOPK_PARAMS,
    K_SORT_COUNT, K_SORT_SCAN, K_SORT_SCATTER, K_SEG_NORMS, K_COUNT
};

constexpr int kTimingPool = 2048;  // event pairs kept between two reads

struct Workspace {
    // per-kernel timing (off by default): one CUDA event pair around every kernel launch
    bool timing;
    int timing_used;
    cudaEvent_t* ev_start;
    cudaEvent_t* ev_stop;
    int* ev_id;
    int64_t launches_by_id[K_COUNT];
    int device;
    int64_t d_max;
    int M_max, L_max;
    int sm_count;
    int64_t launches;
    // device memory
    int* status;                 // sticky status word
    int* worker_err;             // [M] per-worker device error (0 = fine)
    uint32_t* hist1;             // [M][kBins1]  counts, then suffix sums in place
    uint8_t* table1;             // [M][kBins1]  leading-digit bin -> slot of pass 2
    uint32_t* hist2;             // [M][kMaxQueries][256]
    uint8_t* map2;               // [M][kMaxQueries][256] (slot2, digit2) -> slot of pass 3
    uint32_t* hist3;             // [M][kMaxQueries][256]
    Query* queries;              // [M][kMaxQueries]
    double* band_partial;        // [M][norm_ctas][kMaxLevels] per-block open-interval sums (full sweep / bf16)
    int norm_ctas, cur_norm_ctas;
    double* sum_partial;         // [M][sum_ctas][kMaxLevels]  sweep 2: energy of the threshold-free bins
    int sum_ctas, cur_sum_ctas;
    unsigned long long* cand_S;  // [M][kMaxLevels][2 sides][2 halves] integer energy sums of the candidate keys
    uint32_t* cand_keys;         // [M][cand_cap] keys of the boundary-bin elements
    int64_t cand_cap;
    uint32_t* cand_count;        // [M]
    int* cand_overflow;          // [M] 1: the candidates did not fit, full-sweep passes take over
    int64_t* k_dev;              // [kMaxLevels] schedule
    double* p_fixed;             // [kMaxLevels] normalised fixed p
    double* p_all;               // [M][kMaxLevels]
    double* delta_all;           // [M][kMaxLevels]
    double* u_dev;               // [M]
    EmitParams* emit;            // [M]
    uint4* tile_desc;            // [M][tiles per worker] per listed tile {C, A, B}: its own counts, then the running totals before it
    int64_t max_tiles;
    uint32_t* tile_max;          // [M][tiles per worker][kEmitGroups] largest magnitude key of every batch of every emit tile (sweep 1)
    uint32_t* worker_tiles;      // [M][tiles per worker] the tiles of a worker that can hold band entries, ascending: tile | batch mask << 24
    uint32_t* tile_n;            // [M] how many of them
    uint32_t* group_n;           // [M] how many batches they have to read
    int64_t last_emit_tiles;     // tiles per row of the last emission (host side, for mlmc_read_listed_tiles)
    uint32_t* cand_floor;        // [M] smallest key that can be a candidate of sweep 2 (lower edge of the lowest boundary bin)
    uint32_t* agg_offsets;       // [M][agg_tiles_max + 1]
    // bit-wise
    uint32_t* gmax_bits;         // [M]
    unsigned long long* S_partial;  // [M][stat_ctas][kMaxLevels]
    int stat_ctas, cur_stat_ctas;
    int32_t* bit_level;          // [M] (mirrors out->level for the pack kernel)
    // fixed-p Top-k: boundary bins of the previous call, per worker and level boundary, reused as brackets
    uint32_t* prev_bin;          // [M][kMaxLevels] leading-digit bin of threshold j at the last call that resolved it (kKeyNone: none)
    uint4* bracket;              // [M] {lo_a, width_a, lo_b, width_b}: bins collected as candidates by the first sweep
    int* bracket_hit;            // [M] 1: both boundary bins of the drawn band lie in their brackets
    unsigned long long* bracket_stats;  // [3] workers with both brackets hit / a bracket missed / no bracket yet (cumulative)
    int64_t sig_d, sig_ld;       // host: the problem the stored bins belong to
    int sig_M, sig_L, sig_dtype;
    int64_t sig_k[kMaxLevels];
    // s-Top-k with more levels than kMaxLevels (fixed p only): normalised p and its running sums
    double* p_big;               // [big_cap]
    double* cdf_big;             // [big_cap]
    int64_t big_cap;
    uint32_t* sort_scratch;      // key buffers, digit tables and segment norms of the radix sort, for sort_rows rows; allocated at first use
    int sort_rows;               // rows that are sorted together
    // RTN: per-block residual energies of every level
    double* rtn_partial;         // [M][rtn_ctas][kMaxLevels]
    int rtn_ctas, cur_rtn_ctas;
};

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ uint64_t splitmix_finalize(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// One uniform in [0,1) per (seed, step, worker): three chained SplitMix64 output rounds.
__device__ __forceinline__ double counter_uniform(uint64_t seed, uint64_t step, uint64_t worker) {
    const uint64_t golden = 0x9E3779B97F4A7C15ull;
    uint64_t h = splitmix_finalize(seed + golden);
    h = splitmix_finalize(h + step + golden);
    h = splitmix_finalize(h + worker + golden);
    return (double)(h >> 11) * 0x1.0p-53;
}

// cdf in ascending l; the last level with p > 0 and everything after it has cdf 1; l* = min{l : u < cdf_l}
// ("Sample l ~ p^l", Alg. 2 / Alg. 3).
__device__ __forceinline__ int draw_from_probs(const double* p, int L, double u) {
    int j_last = -1;
    for (int j = 0; j < L; ++j)
        if (p[j] > 0.0) j_last = j;
    double c = 0.0;
    for (int j = 0; j < L; ++j) {
        c += p[j];
        const double cdf = (j >= j_last) ? 1.0 : c;
        if (u < cdf) return j;
    }
    return 0;
}

// Magnitude key: monotone in |g| for finite values.  fp32: 31 bits; bf16: 15 bits.
template <typename T>
struct ElemTraits;

template <>
struct ElemTraits<float> {
    static constexpr int kVec = 4;             // elements per 16-byte load
    static constexpr uint32_t kInfKey = 0x7F800000u;
    static constexpr int kShift1 = 16;         // key >> kShift1 = leading digit
    __device__ static __forceinline__ uint32_t key(uint32_t bits) { return bits & 0x7FFFFFFFu; }
    __device__ static __forceinline__ float value(uint32_t bits) { return __uint_as_float(bits); }
};

struct bf16_t {
    uint16_t x;
};

template <>
struct ElemTraits<bf16_t> {
    static constexpr int kVec = 8;
    static constexpr uint32_t kInfKey = 0x7F80u;
    static constexpr int kShift1 = 0;
    __device__ static __forceinline__ uint32_t key(uint32_t bits) { return bits & 0x7FFFu; }
    __device__ static __forceinline__ float value(uint32_t bits) { return __uint_as_float(bits << 16); }
};

// Loads the 16-byte vector v of a row and hands each element's raw bits to f(index_in_row, bits).
// Elements at or past d are skipped; a vector that straddles d is read element by element.
template <typename T, typename F>
__device__ __forceinline__ void for_each_in_vector(const T* row, int64_t v, int64_t d, F&& f) {
    constexpr int V = ElemTraits<T>::kVec;
    const int64_t base = v * V;
    if (base + V <= d) {
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(row) + v);
        if constexpr (V == 4) {
            f(base + 0, q.x);
            f(base + 1, q.y);
            f(base + 2, q.z);
            f(base + 3, q.w);
        } else {
            f(base + 0, q.x & 0xFFFFu);
            f(base + 1, q.x >> 16);
            f(base + 2, q.y & 0xFFFFu);
            f(base + 3, q.y >> 16);
            f(base + 4, q.z & 0xFFFFu);
            f(base + 5, q.z >> 16);
            f(base + 6, q.w & 0xFFFFu);
            f(base + 7, q.w >> 16);
        }
    } else {
        for (int64_t i = base; i < d; ++i) {
            uint32_t bits;
            if constexpr (V == 4)
                bits = reinterpret_cast<const uint32_t*>(row)[i];
            else
                bits = reinterpret_cast<const uint16_t*>(row)[i];
            f(i, bits);
        }
    }
}

// 16-byte asynchronous copy from global to shared memory (cp.async), grouped by commit / wait.
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
    const unsigned sa = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(sa), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// Contiguous range of 16-byte vectors handled by block `bx` of `nb` blocks over a row of d elements.
__device__ __forceinline__ void block_vector_range(int64_t d, int vec, int bx, int nb, int64_t* v0, int64_t* v1) {
    const int64_t nvec = (d + vec - 1) / vec;
    const int64_t per = (nvec + nb - 1) / nb;
    *v0 = min((int64_t)bx * per, nvec);
    *v1 = min(*v0 + per, nvec);
}

// Emit tiles of one row: kEmitTile 32-bit words each (one fp32 or two bf16 elements per word).
inline int emit_tiles_per_worker(int64_t d, int dtype) {
    const int per_word = (dtype == MLMC_BF16) ? 2 : 1;
    const int64_t words = (d + per_word - 1) / per_word;
    return (int)((words + kEmitTile - 1) / kEmitTile);
}

// Brackets one kernel launch: counts it and, when timing is on, records an event pair on the stream.
struct LaunchScope {
    Workspace& ws;
    cudaStream_t s;
    int slot;
    LaunchScope(Workspace& w, int id, cudaStream_t st) : ws(w), s(st), slot(-1) {
        ws.launches++;
        ws.launches_by_id[id]++;
        if (ws.timing && ws.timing_used < kTimingPool) {
            slot = ws.timing_used++;
            ws.ev_id[slot] = id;
            cudaEventRecord(ws.ev_start[slot], s);
        }
    }
    ~LaunchScope() {
        if (slot >= 0) cudaEventRecord(ws.ev_stop[slot], s);
    }
};

// ---------------------------------------------------------------------------------------------
// launchers (each enqueues on `s` and bumps ws.launches)
// ---------------------------------------------------------------------------------------------
// topk_select.cu
int configure_select_kernels();
void launch_init_queries_adaptive(Workspace& ws, int M, int L, int64_t d, cudaStream_t s);
void launch_draw_fixed(Workspace& ws, int M, int L, int64_t d, uint64_t seed, uint64_t step, bool brackets,
                       cudaStream_t s);
void launch_uniforms(Workspace& ws, int M, uint64_t seed, uint64_t step, cudaStream_t s);
void launch_reset_selection(Workspace& ws, int dtype, int64_t d, int M, cudaStream_t s);
void launch_hist1(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, bool brackets, cudaStream_t s);
void launch_resolve1(Workspace& ws, int dtype, int M, int L, bool brackets, cudaStream_t s);
void launch_sums_candidates(Workspace& ws, const void* g, int64_t d, int M, int64_t ld, int L, bool sums,
                            bool brackets, cudaStream_t s);
void launch_digit_pass(Workspace& ws, const void* g, int64_t d, int M, int64_t ld, int pass, cudaStream_t s);
void launch_resolve23(Workspace& ws, int M, int L, int pass, cudaStream_t s);
void launch_band_norms_fp32(Workspace& ws, const void* g, int64_t d, int M, int64_t ld, int L, cudaStream_t s);
void launch_norm_from_hist_bf16(Workspace& ws, int M, int L, cudaStream_t s);
void launch_probs_draw(Workspace& ws, int dtype, int M, int L, int64_t d, bool adaptive, bool want_emit,
                       uint64_t seed, uint64_t step, const mlmc_topk_msgs* out, cudaStream_t s);
void launch_copy_probs(Workspace& ws, int M, int L, const double* p_fixed, double* p_out, double* delta_out,
                       cudaStream_t s);
// topk_emit.cu
int configure_emit_kernels();
void launch_emit(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const mlmc_topk_msgs& out,
                 cudaStream_t s);
void launch_aggregate_topk(Workspace& ws, const mlmc_topk_msgs& msgs, int M, int64_t d, float* out, cudaStream_t s);
// bitwise.cu
int configure_bit_kernels();
void launch_absmax(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, cudaStream_t s);
void launch_bit_stats(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* b, int L,
                      cudaStream_t s);
void launch_bit_probs_draw(Workspace& ws, int M, const int32_t* b, int L, bool adaptive, bool need_delta,
                           uint64_t seed, uint64_t step, const mlmc_bit_msgs* out, cudaStream_t s);
void launch_bit_pack(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* b, int L,
                     const mlmc_bit_msgs& out, cudaStream_t s);
void launch_aggregate_bitwise(Workspace& ws, const mlmc_bit_msgs& msgs, const int32_t* b, int L, int M, int64_t d,
                              float* out, cudaStream_t s);

// floatbits.cu
void launch_compress_floatbits(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* mb,
                               int L, uint64_t seed, uint64_t step, const mlmc_float_msgs& out, cudaStream_t s);
void launch_aggregate_floatbits(Workspace& ws, const mlmc_float_msgs& msgs, const int32_t* mb, int L, int M, int64_t d,
                                float* out, cudaStream_t s);
// rtn.cu
void launch_rtn_stats(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* r, int L,
                      cudaStream_t s);
void launch_rtn_probs_draw(Workspace& ws, int M, int L, bool adaptive, bool have_stats, uint64_t seed, uint64_t step,
                           const mlmc_rtn_msgs* out, cudaStream_t s);
void launch_rtn_emit(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* r, int L,
                     const mlmc_rtn_msgs& out, cudaStream_t s);
void launch_aggregate_dense(Workspace& ws, const float* val, const int32_t* level, int M, int64_t d, int64_t ldv,
                            float* out, cudaStream_t s);
// topk_select.cu: s-Top-k with many levels (fixed p)
void launch_stopk_draw(Workspace& ws, int M, int64_t L, int64_t s_len, int64_t d, uint64_t seed, uint64_t step,
                       cudaStream_t s);
void launch_stopk_params(Workspace& ws, int M, int64_t s_len, int64_t d, const mlmc_topk_msgs* out, cudaStream_t s);
// stopk_sort.cu: s-Top-k with adaptive p and many segments
int configure_sort_kernels();
int stopk_sort_rows(int64_t d_max, int64_t big_cap, int M_max);
size_t stopk_sort_scratch_bytes(int64_t d_max, int64_t big_cap, int M_max);
void launch_stopk_sorted_rows(Workspace& ws, const void* g, int dtype, int64_t d, int m0, int rows, int64_t ld,
                              int64_t s_len, int64_t L, uint64_t seed, uint64_t step, cudaStream_t s);

}  // namespace mlmc
