// Threshold selection, band norms, level probabilities and the level draw for MLMC-Top-k.
//
// The residual C^l(g) - C^{l-1}(g) of Top-k is the band of ranks (k_{l-1}, k_l] of the total order
// (|g| descending, index ascending) (Sec. 3.2).  A band is described by two thresholds: for rank k,
// T = key of the rank-k element, c = #{key > T}, n = #{key == T}, r = k - c = how many of the
// equal-key elements (in index order) are inside Top-k.  Thresholds come from an MSD radix select
// on the magnitude key: a 2^15-bin histogram of the leading digit for all queries at once, then two
// 8-bit digit passes restricted to the boundary bins (fp32 only; a bf16 key is its leading digit).
// With fixed p the level is drawn first; the boundary bins found by one call are the next call's brackets, so
// that the first sweep can collect the boundary-bin keys itself.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kHistThreads = 1024;
constexpr int kResolveThreads = 1024;

// -------------------------------------------------------------------------------------------
// queries
// -------------------------------------------------------------------------------------------
// Adaptive: every level boundary k_0..k_{L-2} is a query.  Fixed p: the level is drawn first
// (it does not depend on the data), and only the two boundaries of its band are live.
__global__ void init_queries_kernel(Query* queries, const int64_t* k, int L, int64_t d, const EmitParams* emit,
                                    int fixed, const uint32_t* prev_bin, uint4* bracket) {
    const int m = blockIdx.x;
    const int j = threadIdx.x;
    if (fixed && bracket && j == 0) {
        // brackets of the first sweep: the bin where each boundary of the drawn band was found last time, and its
        // two neighbours (an empty bracket is {lo = all ones, width = 0}: bin - lo wraps to bin + 1 > 0)
        const int lv = emit[m].level;
        uint4 b = make_uint4(0xFFFFFFFFu, 0u, 0xFFFFFFFFu, 0u);
        if (lv >= 1) {
            const uint32_t pb = prev_bin[m * kMaxLevels + lv - 1];
            if (pb != kKeyNone) { b.x = pb ? pb - 1u : 0u; b.y = pb ? 2u : 1u; }
        }
        if (lv < L - 1) {
            const uint32_t pb = prev_bin[m * kMaxLevels + lv];
            if (pb != kKeyNone) { b.z = pb ? pb - 1u : 0u; b.w = pb ? 2u : 1u; }
        }
        bracket[m] = b;
    }
    if (j >= L - 1) return;
    Query q = {};
    const int64_t kj = k[j];
    q.k = (uint32_t)kj;
    q.slot = kNoSlot;
    q.trivial = (kj <= 0) ? 1u : (kj >= d ? 2u : 0u);
    if (fixed) {
        const int lv = emit[m].level;
        if (j != lv && j != lv - 1) q.trivial = 3u;
    }
    if (q.trivial == 1u || q.trivial == 3u) {
        q.T = kKeyNone;
    } else if (q.trivial == 2u) {
        q.T = 0u;
        q.r = 0xFFFFFFFFu;
    }
    queries[m * kMaxQueries + j] = q;
}

// cdf in ascending l; the last level with p > 0 and everything after it has cdf 1; l* = min{l : u < cdf_l}.
__device__ int draw_level(const double* p, int L, double u) {
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

__global__ void draw_fixed_kernel(const double* p_fixed, int L, uint64_t seed, uint64_t step, double* p_all,
                                  double* u_dev, EmitParams* emit, int M) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    const double u = counter_uniform(seed, step, (uint64_t)m);
    u_dev[m] = u;
    for (int l = 0; l < L; ++l) p_all[m * kMaxLevels + l] = p_fixed[l];
    emit[m].level = draw_level(p_fixed, L, u);
}

__global__ void uniforms_kernel(double* u_dev, int M, uint64_t seed, uint64_t step) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < M) u_dev[m] = counter_uniform(seed, step, (uint64_t)m);
}

// -------------------------------------------------------------------------------------------
// sweep 1: leading-digit histogram of every worker (shared-memory counts, flushed with atomics)
// -------------------------------------------------------------------------------------------
// The sweep also records the largest key of every batch of the emit tiles (kEmitGroupVecs consecutive 16-byte
// vectors of the row): the emit sweep reads only the batches whose largest key reaches the lower threshold of the
// drawn band.  Chunks start at a multiple of 32 vectors, so the 32 vectors a warp loads together lie in one batch.
// BR (fp32, fixed p): the keys whose leading digit lies in one of the worker's two brackets (the bins around last
// call's boundary bins) are collected as candidates in the same sweep.  Every warp stages them in a private
// shared-memory buffer, in lane order by a warp scan, and moves the buffer to the candidate list when it fills up
// (one global counter update per move).
constexpr int kWarpStage = 767;  // keys per warp stage (a warp adds at most 512 per trip), plus one word for its count: 96 KB per block

template <typename T, bool BR>
__global__ void __launch_bounds__(kHistThreads, 1)
hist1_kernel(const T* __restrict__ g, int64_t d, int64_t ld, uint32_t* __restrict__ hist1,
             uint32_t* __restrict__ tile_max, int tiles_per_worker, int* status, int* worker_err,
             const uint4* __restrict__ bracket, uint32_t* __restrict__ cand_keys, int64_t cand_cap,
             uint32_t* cand_count, int* cand_overflow) {
    extern __shared__ uint32_t sh_hist[];
    using Tr = ElemTraits<T>;
    const int m = blockIdx.y;
    // BR only: the warp's stage, its fill count in the word before it
    uint32_t* wcount = sh_hist + kBins1 + (threadIdx.x >> 5) * (kWarpStage + 1);
    uint32_t* wstage = wcount + 1;
    uint32_t lo_a = 0xFFFFFFFFu, span_a = 0u, lo_b = 0xFFFFFFFFu, span_b = 0u;  // key ranges of the two brackets
    if (BR) {
        const uint4 br = bracket[m];
        if (br.x != 0xFFFFFFFFu) { lo_a = br.x << 16; span_a = ((br.y + 1u) << 16) - 1u; }
        if (br.z != 0xFFFFFFFFu) { lo_b = br.z << 16; span_b = ((br.w + 1u) << 16) - 1u; }
        if ((threadIdx.x & 31) == 0) *wcount = 0u;
    }
    const uint32_t lo_min = min(lo_a, lo_b);
    auto in_bracket = [&](uint32_t bits) -> bool {
        const uint32_t key = bits & 0x7FFFFFFFu;
        return (key - lo_a) <= span_a || (key - lo_b) <= span_b;  // an empty bracket: key - lo wraps to key + 1 > 0
    };
    auto flush_stage = [&]() {  // called by the whole warp, after a __syncwarp
        const uint32_t wfill = *wcount;
        if (wfill) {
            uint32_t base = 0;
            if ((threadIdx.x & 31) == 0) base = atomicAdd(&cand_count[m], wfill);
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            if ((int64_t)base + wfill <= cand_cap) {
                uint32_t* dst = cand_keys + (int64_t)m * cand_cap + base;
                for (uint32_t i = threadIdx.x & 31; i < wfill; i += 32) dst[i] = wstage[i];
            } else if ((threadIdx.x & 31) == 0) {
                cand_overflow[m] = 1;
            }
            __syncwarp();
            if ((threadIdx.x & 31) == 0) *wcount = 0u;
            __syncwarp();
        }
    };
    for (int b = threadIdx.x; b < kBins1; b += blockDim.x) sh_hist[b] = 0;
    __syncthreads();
    const T* row = g + (int64_t)m * ld;
    uint32_t* tmax = tile_max + (int64_t)m * tiles_per_worker * kEmitGroups;  // one slot per batch of kEmitGroupVecs vectors
    const int64_t nvec = (d + Tr::kVec - 1) / Tr::kVec;
    bool bad = false;
    auto count_key = [&](uint32_t bits) { atomicAdd(&sh_hist[Tr::key(bits) >> Tr::kShift1], 1u); };  // Inf / NaN: see the maxima
    auto vector_max = [&](const uint4& q) -> uint32_t {  // largest key of one vector
        if constexpr (Tr::kVec == 4) {
            return max(max(q.x & 0x7FFFFFFFu, q.y & 0x7FFFFFFFu), max(q.z & 0x7FFFFFFFu, q.w & 0x7FFFFFFFu));
        } else {
            const uint32_t a = __vmaxu2(__vmaxu2(q.x & 0x7FFF7FFFu, q.y & 0x7FFF7FFFu),
                                        __vmaxu2(q.z & 0x7FFF7FFFu, q.w & 0x7FFF7FFFu));
            return max(a & 0xFFFFu, a >> 16);
        }
    };
    // four 16-byte loads per thread are issued before any of them is used: 64 KB in flight per SM
    constexpr int kBatch = 4;
    const int64_t full_end = d / Tr::kVec;  // vectors that lie wholly inside the row
    const int lane = threadIdx.x & 31;
    // Chunks of kBatch * blockDim.x vectors are dealt round-robin to the blocks of a worker (how fast a chunk is
    // counted depends on how its keys collide in the shared-memory histogram, which differs from layer to layer).
    const int64_t chunk = (int64_t)kBatch * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * chunk; base < nvec; base += (int64_t)gridDim.x * chunk) {
        const int64_t v = base + threadIdx.x;
        if (base + chunk > full_end) {  // the row's last chunk: vector by vector (block-uniform branch)
            for (int64_t u = v; u < nvec; u += blockDim.x) {
                uint32_t vm = 0;
                for_each_in_vector<T>(row, u, d, [&](int64_t, uint32_t bits) {
                    count_key(bits);
                    vm = max(vm, Tr::key(bits));
                    if (BR && in_bracket(bits)) {  // the ragged end of the row: one by one
                        const uint32_t at = atomicAdd(&cand_count[m], 1u);
                        if ((int64_t)at < cand_cap) cand_keys[(int64_t)m * cand_cap + at] = bits & 0x7FFFFFFFu;
                        else cand_overflow[m] = 1;
                    }
                });
                bad |= vm >= Tr::kInfKey;
                atomicMax(&tmax[u / kEmitGroupVecs], vm);
            }
            break;
        }
        uint4 q[kBatch];
        uint32_t vmax[kBatch];  // BR only
#pragma unroll
        for (int j = 0; j < kBatch; ++j) q[j] = __ldg(reinterpret_cast<const uint4*>(row) + v + (int64_t)j * blockDim.x);
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            if constexpr (Tr::kVec == 4) {
                count_key(q[j].x); count_key(q[j].y); count_key(q[j].z); count_key(q[j].w);
            } else {
                count_key(q[j].x & 0xFFFFu); count_key(q[j].x >> 16); count_key(q[j].y & 0xFFFFu); count_key(q[j].y >> 16);
                count_key(q[j].z & 0xFFFFu); count_key(q[j].z >> 16); count_key(q[j].w & 0xFFFFu); count_key(q[j].w >> 16);
            }
            const uint32_t vm = vector_max(q[j]);
            if (BR) vmax[j] = vm;
            const uint32_t wm = __reduce_max_sync(0xFFFFFFFFu, vm);
            bad |= wm >= Tr::kInfKey;  // a non-finite entry shows in the largest key of its warp
            if (lane == 0) atomicMax(&tmax[(v + (int64_t)j * blockDim.x) / kEmitGroupVecs], wm);
        }
        if constexpr (BR) {
            uint32_t cm = 0;  // bit 4 j + e: element e of vector j lies in a bracket
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                if (vmax[j] >= lo_min) {  // a vector whose largest key lies below both brackets holds none of their keys
                    cm |= in_bracket(q[j].x) ? (1u << (4 * j)) : 0u;
                    cm |= in_bracket(q[j].y) ? (2u << (4 * j)) : 0u;
                    cm |= in_bracket(q[j].z) ? (4u << (4 * j)) : 0u;
                    cm |= in_bracket(q[j].w) ? (8u << (4 * j)) : 0u;
                }
            }
            if (cm) {  // this lane's keys go to the warp's stage at a position taken from the warp's counter
                uint32_t pos = atomicAdd(wcount, (uint32_t)__popc(cm));
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    if (cm & (1u << (4 * j))) wstage[pos++] = q[j].x & 0x7FFFFFFFu;
                    if (cm & (2u << (4 * j))) wstage[pos++] = q[j].y & 0x7FFFFFFFu;
                    if (cm & (4u << (4 * j))) wstage[pos++] = q[j].z & 0x7FFFFFFFu;
                    if (cm & (8u << (4 * j))) wstage[pos++] = q[j].w & 0x7FFFFFFFu;
                }
            }
            __syncwarp();
            if (*wcount > (uint32_t)(kWarpStage - 32 * 4 * kBatch)) flush_stage();  // room for one more trip
        }
    }
    if (BR) {
        __syncwarp();
        flush_stage();
    }
    if (bad) {
        worker_err[m] = MLMC_ERR_NONFINITE;
        set_status(status, MLMC_ERR_NONFINITE);
    }
    __syncthreads();
    uint32_t* out = hist1 + (int64_t)m * kBins1;
    for (int b = threadIdx.x; b < kBins1; b += blockDim.x) {
        const uint32_t c = sh_hist[b];
        if (c) atomicAdd(&out[b], c);
    }
}

// -------------------------------------------------------------------------------------------
// block-level helpers for the per-worker resolve kernels
// -------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t warp_inclusive_sum(uint32_t x) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
        if (lane >= o) x += y;
    }
    return x;
}

// Assigns histogram slots to live queries: queries whose fixed prefix (>> shift) agree share a slot.
__device__ void assign_slots(Query* q, int nq, int shift) {
    int next = 0;
    for (int j = 0; j < nq; ++j) {
        if (q[j].trivial) continue;
        int s = -1;
        for (int i = 0; i < j; ++i)
            if (!q[i].trivial && (q[i].prefix >> shift) == (q[j].prefix >> shift)) {
                s = (int)q[i].slot;
                break;
            }
        q[j].slot = (s >= 0) ? (uint32_t)s : (uint32_t)next++;
    }
}

// After sweep 1: suffix sums of the leading-digit histogram in place (S[b] = #{digit >= b}), then
// every live query descends into its bin.  For bf16 the digit is the whole key, so the query is resolved.
// For fp32 the kernel also writes the bin table of the second sweep: a bin that holds no threshold maps
// to its open interval  #{ j : bin_j > b }  (code < 64); a bin that holds one maps to 64 + its slot.
__global__ void __launch_bounds__(kResolveThreads, 1)
resolve1_kernel(uint32_t* hist1, Query* queries, uint8_t* table1, uint32_t* cand_floor, int nq, int is_bf16,
                const int* worker_err, const EmitParams* emit, const uint4* bracket, int* bracket_hit,
                uint32_t* prev_bin, unsigned long long* bracket_stats, uint32_t* cand_count, int* cand_overflow) {
    __shared__ uint32_t sh_warp[32];
    __shared__ uint32_t sh_tot[kResolveThreads], sh_off[kResolveThreads];
    __shared__ int sh_bin[kMaxQueries];
    __shared__ uint32_t sh_slot[kMaxQueries];
    __shared__ bool sh_live[kMaxQueries];
    const int m = blockIdx.x;
    uint32_t* S = hist1 + (int64_t)m * kBins1;
    Query* q = queries + m * kMaxQueries;
    constexpr int per = kBins1 / kResolveThreads;  // 32 chunks of 1024 bins; thread t owns bin c * 1024 + t of chunk c
    static_assert(per == 32 && kResolveThreads == 1024, "the (chunk, warp) totals are scanned by one thread each");
    {
        // suffix sums S[b] = #{digit >= b}, coalesced: 32 chunks of 1024 bins, thread t owns bin c * 1024 + t of
        // chunk c.  Every warp first scans its 32 bins of every chunk, then one scan over the 32 x 32 (chunk, warp)
        // totals gives each of them what lies above it: three barriers in all.
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        uint32_t cnt[per];
#pragma unroll
        for (int c = 0; c < per; ++c) cnt[c] = S[c * kResolveThreads + threadIdx.x];  // all 32 loads in flight at once
#pragma unroll
        for (int c = 0; c < per; ++c) {
            uint32_t v = cnt[c];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {  // inclusive suffix within the warp
                const uint32_t y = __shfl_down_sync(0xFFFFFFFFu, v, o);
                if (lane + o < 32) v += y;
            }
            cnt[c] = v;
            if (lane == 0) sh_tot[c * 32 + warp] = v;
        }
        __syncthreads();
        // entry e = chunk * 32 + warp, taken by thread e: exclusive suffix sum over the entries in that order
        const uint32_t x = sh_tot[threadIdx.x];
        uint32_t v = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_down_sync(0xFFFFFFFFu, v, o);
            if (lane + o < 32) v += y;
        }
        if (lane == 0) sh_warp[warp] = v;  // total of chunk `warp`
        __syncthreads();
        uint32_t higher = 0;
#pragma unroll 8
        for (int c = 0; c < 32; ++c)
            if (c > warp) higher += sh_warp[c];
        sh_off[threadIdx.x] = v - x + higher;
        __syncthreads();
#pragma unroll
        for (int c = 0; c < per; ++c) S[c * kResolveThreads + threadIdx.x] = cnt[c] + sh_off[c * 32 + warp];
    }
    __syncthreads();
    if (worker_err[m]) return;
    {
        // Warp j descends query j: the largest bin b with S[b] >= k (S[0] = d >= k).  S at the first bin of each of
        // the 1024 groups of 32 bins is still in shared memory (group total + what lies above it), so two 32-way
        // votes find the group and one coalesced row of S from memory finds the bin.
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (warp < nq && !q[warp].trivial) {
            Query& qq = q[warp];
            const uint32_t k = qq.k;
            auto group_S = [&](int e) -> uint32_t { return sh_tot[e] + sh_off[e]; };
            uint32_t mk = __ballot_sync(0xFFFFFFFFu, group_S(lane * 32) >= k);
            const int coarse = 31 - __clz((int)mk);   // lane 0 always votes yes
            mk = __ballot_sync(0xFFFFFFFFu, group_S(coarse * 32 + lane) >= k);
            const int e = coarse * 32 + (31 - __clz((int)mk));
            const uint32_t sb = S[e * 32 + lane];
            mk = __ballot_sync(0xFFFFFFFFu, sb >= k);
            const int in_group = 31 - __clz((int)mk);
            const int lo = e * 32 + in_group;
            const uint32_t next_in = __shfl_sync(0xFFFFFFFFu, sb, (in_group + 1) & 31);
            const uint32_t s_lo = __shfl_sync(0xFFFFFFFFu, sb, in_group);
            const uint32_t ab = (lo == kBins1 - 1) ? 0u : (in_group < 31 ? next_in : group_S(e + 1));
            if (lane == 0) {
                if (is_bf16) {
                    qq.T = (uint32_t)lo;
                    qq.c = ab;
                    qq.n = s_lo - ab;
                    qq.r = k - ab;
                } else {
                    qq.prefix = (uint32_t)lo << 16;
                    qq.rem = k - ab;
                }
            }
        }
    }
    __syncthreads();
    if (is_bf16) return;
    if (threadIdx.x < nq) {
        const Query& qq = q[threadIdx.x];
        // trivial queries: "nothing inside" sits above every bin, "everything inside" below every bin
        sh_bin[threadIdx.x] = (qq.trivial == 2u) ? -1 : (qq.trivial ? kBins1 : (int)(qq.prefix >> 16));
        sh_live[threadIdx.x] = qq.trivial == 0u;
    }
    __syncthreads();
    if (threadIdx.x == 0) {  // slots of the second digit pass: live queries in the same bin share one
        int next = 0;
        for (int jq = 0; jq < nq; ++jq) {
            sh_slot[jq] = kNoSlot;
            if (!sh_live[jq]) continue;
            int sl = -1;
            for (int i = 0; i < jq; ++i)
                if (sh_live[i] && sh_bin[i] == sh_bin[jq]) { sl = (int)sh_slot[i]; break; }
            sh_slot[jq] = (sl >= 0) ? (uint32_t)sl : (uint32_t)next++;
        }
    }
    __syncthreads();
    if (threadIdx.x < nq && sh_live[threadIdx.x]) q[threadIdx.x].slot = sh_slot[threadIdx.x];
    if (threadIdx.x == 0) {
        // the smallest key that can be a candidate: the lower edge of the lowest boundary bin (no live query: none)
        int lowest = kBins1;
        for (int j = 0; j < nq; ++j)
            if (sh_bin[j] >= 0 && sh_bin[j] < lowest) lowest = sh_bin[j];
        cand_floor[m] = (lowest < kBins1) ? ((uint32_t)lowest << 16) : 0xFFFFFFFFu;
        if (bracket) {
            // Did the first sweep already collect the keys of every boundary bin?  (fixed p: the live queries are
            // the boundaries level - 1 and level of the drawn band.)  If not, its candidates are dropped and the
            // candidate sweep runs.  Either way the bins are remembered for the next call.
            const uint4 br = bracket[m];
            const int lv = emit[m].level;
            bool hit = cand_overflow[m] == 0, had = false;
            for (int j = 0; j < nq; ++j) {
                if (q[j].trivial) continue;
                const uint32_t bin = (uint32_t)sh_bin[j];
                const bool a = (j == lv - 1), inside = a ? (bin - br.x) <= br.y : (bin - br.z) <= br.w;
                had |= (a ? br.x : br.z) != 0xFFFFFFFFu;
                hit &= inside;
                prev_bin[m * kMaxLevels + j] = bin;
            }
            bracket_hit[m] = hit ? 1 : 0;
            if (!hit) {
                cand_count[m] = 0u;
                cand_overflow[m] = 0;
            }
            atomicAdd(&bracket_stats[hit ? 0 : (had ? 1 : 2)], 1ull);
        }
    }
    // code of bin b: the number of leading queries whose bin lies above b, or 64 + slot if the first one that does
    // not lies in b itself.  That number can only grow as b falls, so the thread walks its bins downwards.
    uint8_t* tab = table1 + (int64_t)m * kBins1;
    int j = 0;
    for (int i = per - 1; i >= 0; --i) {
        const int b = i * kResolveThreads + threadIdx.x;
        while (j < nq && sh_bin[j] > b) ++j;
        tab[b] = (uint8_t)((j < nq && sh_bin[j] == b) ? 64u + sh_slot[j] : (uint32_t)j);
    }
}

// -------------------------------------------------------------------------------------------
// sweep 2 (fp32): per-interval energy of the bins that hold no threshold, and compaction of the keys
// of the bins that do ("candidates": a few percent of the data) for the remaining digit passes
// -------------------------------------------------------------------------------------------
constexpr int kS2Threads = 512;
constexpr int kS2Vecs = 2;                                   // 16-byte vectors per thread per round
constexpr int kS2Round = kS2Threads * kS2Vecs * 4;            // elements per round
constexpr int kStageSlack = 1024;                             // candidates that may wait for the next flush
constexpr int kStage = kS2Round + kStageSlack;                // staged candidate keys per block

// table: bin -> code.  code < 64: the bin lies wholly inside open interval `code` (between two thresholds);
// code >= 64: the bin may hold a threshold, its keys are compacted into the candidate buffer.
// SUMS: per-interval energy of the threshold-free bins (adaptive p).  Loads are double-buffered in registers:
// the next round's 16-byte vectors are in flight while the current round is processed.
template <bool SUMS>
__global__ void __launch_bounds__(kS2Threads, 2)
sums_candidates_kernel(const float* __restrict__ g, int64_t d, int64_t ld, const uint8_t* __restrict__ table, int L,
                       double* __restrict__ sum_partial, int sum_ctas,
                       uint32_t* __restrict__ cand_keys, int64_t cand_cap, uint32_t* cand_count, int* cand_overflow,
                       const int* worker_err, const uint32_t* __restrict__ tile_max,
                       int tiles_per_worker, const uint32_t* __restrict__ cand_floor,
                       const int* __restrict__ bracket_hit) {
    extern __shared__ __align__(16) uint8_t sh_raw[];
    uint8_t* sh_table = sh_raw;                                                   // [32768]
    uint32_t* sh_stage = reinterpret_cast<uint32_t*>(sh_raw + kBins1);            // [kStage]
    double* sh_acc = reinterpret_cast<double*>(sh_raw + kBins1 + kStage * 4);     // [L][kS2Threads]  (SUMS)
    __shared__ uint32_t sh_n;
    __shared__ uint32_t sh_base;
    const int m = blockIdx.y;
    if (worker_err[m]) return;
    if (!SUMS && bracket_hit && bracket_hit[m]) return;  // the first sweep collected every boundary-bin key already
    {
        const uint4* src = reinterpret_cast<const uint4*>(table + (int64_t)m * kBins1);
        uint4* dst = reinterpret_cast<uint4*>(sh_table);
        for (int i = threadIdx.x; i < kBins1 / 16; i += kS2Threads) dst[i] = src[i];
        if (SUMS)
            for (int i = threadIdx.x; i < L * kS2Threads; i += kS2Threads) sh_acc[i] = 0.0;
        if (threadIdx.x == 0) sh_n = 0;
    }
    __syncthreads();
    const float* row = g + (int64_t)m * ld;
    uint32_t* cand = cand_keys + (int64_t)m * cand_cap;
    // A round is one emit tile (kEmitTileVecs vectors); block b takes rounds b, b + gridDim.x, ...  Without
    // energies (fixed p) only the candidates matter: a tile whose largest key lies below the lowest boundary bin
    // holds none and is not read.  Such tiles cluster (whole layers lie below the thresholds), so the rounds are
    // dealt out round-robin rather than in contiguous ranges.
    static_assert(kS2Threads * kS2Vecs == kEmitTileVecs, "one round of the sweep is one emit tile");
    const int64_t v1 = (d + 3) / 4;                                  // vectors of the row
    const int64_t v0 = min((int64_t)blockIdx.x * kEmitTileVecs, v1);  // this block's first round
    const int64_t vstep = (int64_t)gridDim.x * kEmitTileVecs;
    const int64_t full_end = d / 4;  // vectors wholly inside the row
    // which of the block's rounds hold a candidate, looked up once (rounds past the flag array are swept anyway)
    constexpr int kWantFlags = 2048;
    __shared__ uint8_t sh_want[kWantFlags];
    if (!SUMS) {
        const uint32_t floor_key = cand_floor[m];
        const uint4* tmax = reinterpret_cast<const uint4*>(tile_max + ((int64_t)m * tiles_per_worker + blockIdx.x) * kEmitGroups);
        const int64_t nrounds = (v1 - v0 + vstep - 1) / vstep;
        static_assert(kEmitGroups == 8, "a tile's batch maxima are two 16-byte vectors");
        for (int r = threadIdx.x; r < kWantFlags && r < nrounds; r += kS2Threads) {
            const uint4 a = tmax[(int64_t)r * gridDim.x * 2], b = tmax[(int64_t)r * gridDim.x * 2 + 1];
            sh_want[r] = max(max(max(a.x, a.y), max(a.z, a.w)), max(max(b.x, b.y), max(b.z, b.w))) >= floor_key;
        }
        __syncthreads();
    }
    auto wanted = [&](int64_t vb) -> bool {  // block-uniform
        if (SUMS) return true;
        const int64_t r = (vb - v0) / vstep;
        return vb < v1 && (r >= kWantFlags || sh_want[r]);
    };

    auto flush = [&]() {  // called by all threads
        const uint32_t n = sh_n;
        if (threadIdx.x == 0 && n) sh_base = atomicAdd(&cand_count[m], n);
        __syncthreads();
        if (n) {
            const uint32_t base = sh_base;
            if ((int64_t)base + n <= cand_cap) {
                for (uint32_t i = threadIdx.x; i < n; i += kS2Threads) cand[base + i] = sh_stage[i];
            } else if (threadIdx.x == 0) {
                cand_overflow[m] = 1;  // too many keys share the boundary bins: the full-sweep passes take over
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) sh_n = 0;
        __syncthreads();
    };
    // One element: its energy goes to the interval's accumulator; a key of a boundary bin only sets its bit in `cm`,
    // and the thread stages all its candidates of the round together (one counter update and one divergent region
    // per thread and round instead of one per candidate).
    auto take = [&](uint32_t bits, uint32_t bit, uint32_t& cm) {
        const uint32_t key = bits & 0x7FFFFFFFu;
        const uint32_t code = sh_table[key >> 16];
        if (code < 64u) {
            if (SUMS) {
                const double x = (double)__uint_as_float(key);
                double* a = &sh_acc[code * kS2Threads + threadIdx.x];
                *a = fma(x, x, *a);
            }
        } else {
            cm |= bit;
        }
    };
    auto load_round = [&](int64_t vb, uint4 (&q)[kS2Vecs]) {
#pragma unroll
        for (int j = 0; j < kS2Vecs; ++j) {
            const int64_t v = vb + j * kS2Threads + threadIdx.x;
            if (v < full_end) q[j] = __ldg(reinterpret_cast<const uint4*>(row) + v);
        }
    };

    uint4 cur[kS2Vecs], nxt[kS2Vecs];
    bool want_cur = wanted(v0);
    if (want_cur) load_round(v0, cur);
    for (int64_t vb = v0; vb < v1; vb += vstep) {
        const bool want_nxt = wanted(vb + vstep);
        if (want_nxt) load_round(vb + vstep, nxt);
        if (!SUMS && !want_cur) {  // nothing to do in this round: no barrier either (block-uniform)
            want_cur = want_nxt;
#pragma unroll
            for (int j = 0; j < kS2Vecs; ++j) cur[j] = nxt[j];
            continue;
        }
        uint32_t cm = 0;  // bit 4 j + e: element e of vector j is a candidate
#pragma unroll
        for (int j = 0; j < kS2Vecs; ++j) {
            const int64_t v = vb + j * kS2Threads + threadIdx.x;
            if (v < full_end) {
                take(cur[j].x, 1u << (4 * j), cm); take(cur[j].y, 2u << (4 * j), cm);
                take(cur[j].z, 4u << (4 * j), cm); take(cur[j].w, 8u << (4 * j), cm);
            } else if (v < v1) {  // ragged tail of the row: staged one by one
                for (int64_t i = v * 4; i < d; ++i) {
                    uint32_t one = 0;
                    const uint32_t bits = reinterpret_cast<const uint32_t*>(row)[i];
                    take(bits, 1u, one);
                    if (one) sh_stage[atomicAdd(&sh_n, 1u)] = bits & 0x7FFFFFFFu;
                }
            }
        }
        if (cm) {
            uint32_t pos = atomicAdd(&sh_n, (uint32_t)__popc(cm));
#pragma unroll
            for (int j = 0; j < kS2Vecs; ++j) {
                if (cm & (1u << (4 * j))) sh_stage[pos++] = cur[j].x & 0x7FFFFFFFu;
                if (cm & (2u << (4 * j))) sh_stage[pos++] = cur[j].y & 0x7FFFFFFFu;
                if (cm & (4u << (4 * j))) sh_stage[pos++] = cur[j].z & 0x7FFFFFFFu;
                if (cm & (8u << (4 * j))) sh_stage[pos++] = cur[j].w & 0x7FFFFFFFu;
            }
        }
        __syncthreads();
        if (sh_n > (uint32_t)kStageSlack) flush();  // uniform: sh_n is read after the barrier; a round adds at most kS2Round
        want_cur = want_nxt;
#pragma unroll
        for (int j = 0; j < kS2Vecs; ++j) cur[j] = nxt[j];
    }
    flush();
    if (SUMS) {
        for (int l = 0; l < L; ++l) {  // fixed-order tree: reproducible sums
            double* a = sh_acc + l * kS2Threads;
            for (int s = kS2Threads >> 1; s > 0; s >>= 1) {
                if (threadIdx.x < s) a[threadIdx.x] += a[threadIdx.x + s];
                __syncthreads();
            }
            if (threadIdx.x == 0) sum_partial[((int64_t)m * sum_ctas + blockIdx.x) * kMaxLevels + l] = a[0];
        }
    }
}

// Digit pass over the compacted candidate keys (normal case).
template <int PASS>
__device__ __forceinline__ void cand_pass_body(uint32_t* sh_hist, int bx, int nbx, const uint32_t* __restrict__ cand_keys,
                                               int64_t cand_cap, const uint32_t* __restrict__ cand_count,
                                               const int* __restrict__ cand_overflow, const uint8_t* __restrict__ table1,
                                               const uint8_t* __restrict__ map2, uint32_t* __restrict__ hist_out,
                                               const int* worker_err) {
    const int m = blockIdx.y;
    if (worker_err[m] || cand_overflow[m]) return;
    const uint32_t n = cand_count[m];
    if ((uint64_t)bx * kSweepThreads >= n) return;
    for (int i = threadIdx.x; i < kMaxQueries * kBins23; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    const uint32_t* cand = cand_keys + (int64_t)m * cand_cap;
    const uint8_t* tab = table1 + (int64_t)m * kBins1;
    const uint8_t* mp = map2 + (int64_t)m * kMaxQueries * kBins23;
    for (uint32_t i = bx * blockDim.x + threadIdx.x; i < n; i += nbx * blockDim.x) {
        const uint32_t key = cand[i];
        const uint32_t code = __ldg(&tab[key >> 16]);
        if (code < 64u) continue;  // a bracket bin that holds no threshold after all
        const uint32_t s2 = code - 64u;
        if (PASS == 2) {
            atomicAdd(&sh_hist[s2 * kBins23 + ((key >> 8) & 0xFFu)], 1u);
        } else {
            const uint32_t s3 = __ldg(&mp[s2 * kBins23 + ((key >> 8) & 0xFFu)]);
            if (s3 != kNoSlot) atomicAdd(&sh_hist[s3 * kBins23 + (key & 0xFFu)], 1u);
        }
    }
    __syncthreads();
    uint32_t* out = hist_out + (int64_t)m * kMaxQueries * kBins23;
    for (int i = threadIdx.x; i < kMaxQueries * kBins23; i += blockDim.x) {
        const uint32_t c = sh_hist[i];
        if (c) atomicAdd(&out[i], c);
    }
}

// Energy of the candidate keys per open interval, now that the thresholds are exact.
// The candidate buffer is filled in an order that changes from run to run, so the sums are taken in
// integers, where the order does not matter: every candidate lies in a boundary bin, all keys of one
// bin share their exponent, so g^2 = mant^2 * 2^(2 (max(e,1) - 150)) with a 48-bit integer mant^2.
// An open interval (T_l, T_{l-1}) meets at most two boundary bins: the bin of T_{l-1} (side 0) and
// the bin of T_l (side 1).  Per (interval, side) the low and the high 24 bits of mant^2 are added
// separately in u64 (no overflow below 2^40 terms) and combined in 128 bits by the draw kernel.
constexpr int kCandSumThreads = 128;

__global__ void __launch_bounds__(kCandSumThreads)
cand_sums_kernel(const uint32_t* __restrict__ cand_keys, int64_t cand_cap, const uint32_t* __restrict__ cand_count,
                 const int* __restrict__ cand_overflow, const Query* __restrict__ queries, int L,
                 unsigned long long* __restrict__ cand_S, const int* worker_err) {
    extern __shared__ unsigned long long sh_S[];  // [L][4][kCandSumThreads]: (side, half) pairs per interval
    __shared__ uint32_t sh_thr[kMaxQueries];
    const int m = blockIdx.y;
    if (worker_err[m] || cand_overflow[m]) return;
    const uint32_t n = cand_count[m];
    if ((uint64_t)blockIdx.x * kCandSumThreads >= n) return;
    for (int i = threadIdx.x; i < L * 4 * kCandSumThreads; i += kCandSumThreads) sh_S[i] = 0ull;
    if (threadIdx.x < kMaxQueries)
        sh_thr[threadIdx.x] = (threadIdx.x < L - 1) ? queries[m * kMaxQueries + threadIdx.x].T : 0u;
    __syncthreads();
    const uint32_t* cand = cand_keys + (int64_t)m * cand_cap;
    const int nthr = L - 1;
    for (uint32_t i = blockIdx.x * kCandSumThreads + threadIdx.x; i < n; i += gridDim.x * kCandSumThreads) {
        const uint32_t key = cand[i];
        int lo = 0, hi = nthr;  // thresholds are descending: first index with T <= key
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sh_thr[mid] > key) lo = mid + 1; else hi = mid;
        }
        if (lo == nthr || sh_thr[lo] != key) {
            const int side = (lo > 0 && (sh_thr[lo - 1] >> 16) == (key >> 16)) ? 0 : 1;
            const uint64_t mant = (key & 0x7FFFFFu) | ((key >> 23) ? 0x800000u : 0u);
            const uint64_t m2 = mant * mant;
            unsigned long long* a = &sh_S[((lo * 2 + side) * 2) * kCandSumThreads + threadIdx.x];
            a[0] += m2 & 0xFFFFFFull;
            a[kCandSumThreads] += m2 >> 24;
        }
    }
    __syncthreads();
    // each warp adds up every fourth (interval, side, half) column: four values per lane, then a shuffle tree
    unsigned long long* out = cand_S + (int64_t)m * kMaxLevels * 4;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = warp; q < L * 4; q += kCandSumThreads / 32) {
        const unsigned long long* a = sh_S + q * kCandSumThreads;
        unsigned long long x = 0;
#pragma unroll
        for (int i = 0; i < kCandSumThreads / 32; ++i) x += a[i * 32 + lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
        if (lane == 0 && x) atomicAdd(&out[q], x);  // integer: the order of the blocks does not matter
    }
}

// -------------------------------------------------------------------------------------------
// full-sweep digit passes (fp32): only for a worker whose candidate buffer overflowed, i.e. when a
// large share of its entries falls into the boundary bins (many equal magnitudes)
// -------------------------------------------------------------------------------------------
template <int PASS>
__device__ __forceinline__ void masked_pass_body(uint8_t* sh_raw, int bx, int nbx, const float* __restrict__ g, int64_t d,
                                                 int64_t ld, const uint8_t* __restrict__ table1,
                                                 const uint8_t* __restrict__ map2, uint32_t* __restrict__ hist_out,
                                                 const int* worker_err, const int* __restrict__ cand_overflow) {
    uint32_t* sh_hist = reinterpret_cast<uint32_t*>(sh_raw);                        // [32][256]
    uint8_t* sh_table = sh_raw + kMaxQueries * kBins23 * sizeof(uint32_t);          // [32768]
    uint8_t* sh_map = sh_table + kBins1;                                            // [32][256] (pass 3)
    const int m = blockIdx.y;
    if (worker_err[m] || !cand_overflow[m]) return;
    for (int i = threadIdx.x; i < kMaxQueries * kBins23; i += blockDim.x) sh_hist[i] = 0;
    {
        const uint4* src = reinterpret_cast<const uint4*>(table1 + (int64_t)m * kBins1);
        uint4* dst = reinterpret_cast<uint4*>(sh_table);
        for (int i = threadIdx.x; i < kBins1 / 16; i += blockDim.x) dst[i] = src[i];
        if (PASS == 3) {
            const uint4* s2 = reinterpret_cast<const uint4*>(map2 + (int64_t)m * kMaxQueries * kBins23);
            uint4* d2 = reinterpret_cast<uint4*>(sh_map);
            for (int i = threadIdx.x; i < kMaxQueries * kBins23 / 16; i += blockDim.x) d2[i] = s2[i];
        }
    }
    __syncthreads();
    const float* row = g + (int64_t)m * ld;
    int64_t v0, v1;
    block_vector_range(d, 4, bx, nbx, &v0, &v1);
#pragma unroll 4
    for (int64_t v = v0 + threadIdx.x; v < v1; v += blockDim.x) {
        for_each_in_vector<float>(row, v, d, [&](int64_t, uint32_t bits) {
            const uint32_t key = bits & 0x7FFFFFFFu;
            const uint32_t code = sh_table[key >> 16];
            if (code >= 64u) {
                const uint32_t s2 = code - 64u;
                if (PASS == 2) {
                    atomicAdd(&sh_hist[s2 * kBins23 + ((key >> 8) & 0xFFu)], 1u);
                } else {
                    const uint32_t s3 = sh_map[s2 * kBins23 + ((key >> 8) & 0xFFu)];
                    if (s3 != kNoSlot) atomicAdd(&sh_hist[s3 * kBins23 + (key & 0xFFu)], 1u);
                }
            }
        });
    }
    __syncthreads();
    uint32_t* out = hist_out + (int64_t)m * kMaxQueries * kBins23;
    for (int i = threadIdx.x; i < kMaxQueries * kBins23; i += blockDim.x) {
        const uint32_t c = sh_hist[i];
        if (c) atomicAdd(&out[i], c);
    }
}

// One launch per digit pass: the first nb_cand blocks of a worker take its compacted candidate keys, the others are
// the full-row fall-back (they return at once unless the worker's candidate buffer overflowed).
template <int PASS>
__global__ void __launch_bounds__(kSweepThreads)
digit_pass_kernel(int nb_cand, const float* __restrict__ g, int64_t d, int64_t ld,
                  const uint32_t* __restrict__ cand_keys, int64_t cand_cap, const uint32_t* __restrict__ cand_count,
                  const int* __restrict__ cand_overflow, const uint8_t* __restrict__ table1,
                  const uint8_t* __restrict__ map2, uint32_t* __restrict__ hist_out, const int* worker_err) {
    extern __shared__ __align__(16) uint8_t sh_digit[];
    if ((int)blockIdx.x < nb_cand)
        cand_pass_body<PASS>(reinterpret_cast<uint32_t*>(sh_digit), blockIdx.x, nb_cand, cand_keys, cand_cap, cand_count,
                             cand_overflow, table1, map2, hist_out, worker_err);
    else
        masked_pass_body<PASS>(sh_digit, blockIdx.x - nb_cand, gridDim.x - nb_cand, g, d, ld, table1, map2, hist_out,
                               worker_err, cand_overflow);
}

// One warp per query walks its 256-bin histogram from the top digit down.
template <int PASS>
__global__ void __launch_bounds__(kResolveThreads, 1)
resolve23_kernel(const uint32_t* hist, Query* queries, uint8_t* map2, int nq, const int* worker_err) {
    const int m = blockIdx.x;
    if (worker_err[m]) return;
    Query* q = queries + m * kMaxQueries;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < nq && !q[warp].trivial) {
        Query& qq = q[warp];
        const uint32_t* h = hist + ((int64_t)m * kMaxQueries + qq.slot) * kBins23;
        // lane 0 owns the top 8 digits (255..248), lane 31 the bottom 8
        uint32_t cnt[8], local = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            cnt[i] = h[255 - (lane * 8 + i)];
            local += cnt[i];
        }
        const uint32_t rem = qq.rem, prefix = qq.prefix;  // read by every lane before the owning lane rewrites them
        const uint32_t inc = warp_inclusive_sum(local);
        const bool mine = (inc >= rem) && (inc - local < rem);
        __syncwarp();
        if (mine) {
            uint32_t above = inc - local;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (above + cnt[i] >= rem) {
                    const uint32_t digit = 255u - (uint32_t)(lane * 8 + i);
                    if (PASS == 2) {
                        qq.prefix = prefix | (digit << 8);
                        qq.rem = rem - above;
                    } else {
                        qq.T = prefix | digit;
                        qq.r = rem - above;
                        qq.n = cnt[i];
                        qq.c = qq.k - qq.r;
                    }
                    break;
                }
                above += cnt[i];
            }
        }
    }
    __syncthreads();
    if (PASS == 2 && threadIdx.x == 0) {
        // remember the pass-2 slot of each query before the slots are reassigned for pass 3
        uint32_t slot2[kMaxQueries];
        for (int j = 0; j < nq; ++j) slot2[j] = q[j].slot;
        assign_slots(q, nq, 8);
        for (int j = 0; j < nq; ++j)
            if (!q[j].trivial)
                map2[((int64_t)m * kMaxQueries + slot2[j]) * kBins23 + ((q[j].prefix >> 8) & 0xFFu)] = (uint8_t)q[j].slot;
    }
}

// -------------------------------------------------------------------------------------------
// band norms by a full sweep (adaptive fp32, only for a worker whose candidate buffer overflowed):
// sum of g^2 over the open key intervals between consecutive thresholds
// -------------------------------------------------------------------------------------------
// Element with key x belongs to open interval b = #{ l : T_l > x } unless x equals a threshold
// (equal-key elements are split between bands by rank; their energy is added from the counts).
// Every thread owns a private fp64 accumulator per interval in shared memory: no atomics, and a
// fixed reduction order, so the sums are reproducible.
__global__ void __launch_bounds__(kSweepThreads)
norm_sweep_kernel(const float* __restrict__ g, int64_t d, int64_t ld, const Query* __restrict__ queries, int L,
                  double* __restrict__ band_partial, int norm_ctas, const int* worker_err,
                  const int* __restrict__ cand_overflow) {
    extern __shared__ double sh_acc[];  // [L][blockDim]
    __shared__ uint32_t sh_thr[kMaxQueries];
    const int m = blockIdx.y;
    if (worker_err[m] || !cand_overflow[m]) return;
    const int nt = blockDim.x;
    for (int i = threadIdx.x; i < L * nt; i += nt) sh_acc[i] = 0.0;
    if (threadIdx.x < kMaxQueries)
        sh_thr[threadIdx.x] = (threadIdx.x < L - 1) ? queries[m * kMaxQueries + threadIdx.x].T : 0u;
    __syncthreads();
    const float* row = g + (int64_t)m * ld;
    int64_t v0, v1;
    block_vector_range(d, 4, blockIdx.x, gridDim.x, &v0, &v1);
    const int nthr = L - 1;
#pragma unroll 2
    for (int64_t v = v0 + threadIdx.x; v < v1; v += nt) {
        for_each_in_vector<float>(row, v, d, [&](int64_t, uint32_t bits) {
            const uint32_t key = bits & 0x7FFFFFFFu;
            // thresholds are descending: b = first index with T_b <= key
            int lo = 0, hi = nthr;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (sh_thr[mid] > key) lo = mid + 1; else hi = mid;
            }
            if (lo == nthr || sh_thr[lo] != key) {
                const double x = (double)__uint_as_float(key);
                double* a = &sh_acc[lo * nt + threadIdx.x];
                *a = fma(x, x, *a);
            }
        });
    }
    __syncthreads();
    // fixed-order tree reduction per interval
    for (int l = 0; l < L; ++l) {
        double* a = sh_acc + l * nt;
        for (int s = nt >> 1; s > 0; s >>= 1) {
            if (threadIdx.x < s) a[threadIdx.x] += a[threadIdx.x + s];
            __syncthreads();
        }
        if (threadIdx.x == 0) band_partial[((int64_t)m * norm_ctas + blockIdx.x) * kMaxLevels + l] = a[0];
    }
}

// bf16: every key is a histogram bin, so the open-interval sums follow from the counts exactly.
// kNormParts blocks per worker, each over a contiguous 1 / kNormParts of the bins; a bin lies in exactly one open
// interval (or is a threshold), found by a search over the thresholds.  Per interval every warp adds up its lanes'
// shares by shuffles; after one barrier thread l adds the warp sums of interval l in warp order, and the draw
// kernel adds the kNormParts partials in block order (fixed orders: reproducible).
constexpr int kNormParts = 8;
constexpr int kNormThreads = 256;

__global__ void __launch_bounds__(kNormThreads)
norm_from_hist_bf16_kernel(const uint32_t* hist1 /* suffix sums */, const Query* queries, int L,
                           double* band_partial, int norm_ctas, const int* worker_err) {
    __shared__ double sh_part[kMaxLevels][kNormThreads / 32];
    __shared__ uint32_t sh_thr[kMaxQueries];
    const int m = blockIdx.y, part = blockIdx.x;
    if (worker_err[m]) return;
    const uint32_t* S = hist1 + (int64_t)m * kBins1;
    if (threadIdx.x < kMaxQueries)
        sh_thr[threadIdx.x] = (threadIdx.x < L - 1) ? queries[m * kMaxQueries + threadIdx.x].T : 0u;
    __syncthreads();
    constexpr int per = kBins1 / kNormParts / kNormThreads;  // 16 bins per thread, coalesced over the block
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nthr = L - 1;
    double e[per];   // energy of this thread's bins
    int iv[per];     // their open interval, or -1 (empty bin, threshold bin: added from the counts by the draw kernel)
#pragma unroll
    for (int i = 0; i < per; ++i) {
        const uint32_t key = (uint32_t)part * (kBins1 / kNormParts) + i * kNormThreads + threadIdx.x;
        const uint32_t cnt = S[key] - ((key == kBins1 - 1) ? 0u : S[key + 1]);
        int lo = 0, hi = nthr;  // thresholds are descending: first index with T <= key
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (sh_thr[mid] > key) lo = mid + 1; else hi = mid;
        }
        const bool is_thr = lo < nthr && sh_thr[lo] == key;
        iv[i] = (cnt == 0u || is_thr) ? -1 : lo;  // empty bins include the Inf/NaN encodings, whose value must not enter the sum
        const double x = (double)__uint_as_float(key << 16);
        e[i] = (double)cnt * (x * x);
    }
    for (int l = 0; l < L; ++l) {
        double acc = 0.0;
#pragma unroll
        for (int i = 0; i < per; ++i)
            if (iv[i] == l) acc += e[i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) sh_part[l][warp] = acc;
    }
    __syncthreads();
    if (threadIdx.x < L) {
        double tot = 0.0;
        for (int w = 0; w < kNormThreads / 32; ++w) tot += sh_part[threadIdx.x][w];
        band_partial[((int64_t)m * norm_ctas + part) * kMaxLevels + threadIdx.x] = tot;
    }
}

// -------------------------------------------------------------------------------------------
// probabilities, draw, emit parameters
// -------------------------------------------------------------------------------------------
__device__ void fill_emit(int m, int level, double p_sel, const Query* q, const int64_t* k, int L, int64_t d,
                          EmitParams* emit, int64_t* out_count, int32_t* out_level, double* out_p_sel,
                          int64_t capacity, int* status, int* worker_err) {
    EmitParams e = {};
    e.level = level;
    if (level == 0) {
        e.Ta = kKeyNone;
        e.ra = 0;
    } else {
        e.Ta = q[level - 1].T;
        e.ra = q[level - 1].r;
    }
    if (level == L - 1) {
        e.Tb = 0u;
        e.rb = 0xFFFFFFFFu;
    } else {
        e.Tb = q[level].T;
        e.rb = q[level].r;
    }
    e.inv_p = (p_sel > 0.0) ? 1.0 / p_sel : 0.0;
    const int64_t lo = level ? k[level - 1] : 0;
    e.expect = (uint32_t)(k[level] - lo);
    e.enabled = 1;
    if ((int64_t)e.expect > capacity) {
        e.enabled = 0;
        worker_err[m] = MLMC_ERR_CAPACITY;
        set_status(status, MLMC_ERR_CAPACITY);
    }
    emit[m] = e;
    out_count[m] = e.enabled ? (int64_t)e.expect : 0;
    out_level[m] = e.enabled ? level : -1;
    out_p_sel[m] = p_sel;
}

__device__ void fail_worker(int m, EmitParams* emit, int64_t* out_count, int32_t* out_level, double* out_p_sel) {
    EmitParams e = {};
    e.level = -1;
    emit[m] = e;
    if (out_count) out_count[m] = 0;
    if (out_level) out_level[m] = -1;
    if (out_p_sel) out_p_sel[m] = 0.0;
}

// One block per worker.  Adaptive: E_l = open-interval sum + sum over distinct threshold keys K of
// |ranks of K  intersect  (k_{l-1}, k_l]| * val(K)^2;  Delta_l = sqrt(E_l);  p_l = Delta_l / sum Delta
// (Lemma 3.4).  Then the level draw and the two thresholds of the drawn band.
__global__ void probs_draw_kernel(const Query* queries, const int64_t* k, int L, int64_t d, int is_bf16,
                                  const double* band_partial, int norm_ctas, int n_band,
                                  const double* sum_partial, int sum_ctas, int n_sum,
                                  const unsigned long long* cand_S,
                                  const int* cand_overflow, int adaptive,
                                  uint64_t seed, uint64_t step, double* p_all, double* delta_all, double* u_dev,
                                  EmitParams* emit, int64_t* out_count, int32_t* out_level, double* out_p_sel,
                                  int64_t capacity, int* status, int* worker_err, int want_emit) {
    __shared__ double sh_delta[kMaxLevels];
    __shared__ double sh_p[kMaxLevels];
    __shared__ uint32_t sh_T[kMaxQueries], sh_c[kMaxQueries], sh_n[kMaxQueries];
    __shared__ bool sh_first[kMaxQueries];  // a live query whose threshold key no earlier live query has
    const int m = blockIdx.x;
    const Query* q = queries + m * kMaxQueries;
    if (worker_err[m]) {
        if (threadIdx.x == 0 && want_emit) fail_worker(m, emit, out_count, out_level, out_p_sel);
        return;
    }
    const int l = threadIdx.x;
    if (adaptive) {
        if (l < L - 1) {
            sh_T[l] = q[l].trivial ? kKeyNone : q[l].T;
            sh_c[l] = q[l].c;
            sh_n[l] = q[l].n;
        }
        __syncwarp();
        if (l < L - 1) {
            bool first = !q[l].trivial;
            for (int i = 0; i < l; ++i) first &= !(sh_T[i] == sh_T[l] && sh_T[i] != kKeyNone);
            sh_first[l] = first;
        }
        __syncwarp();
    }
    if (adaptive && l < L) {
        // open-interval energy: per-block partials added in block order (reproducible).
        // bf16 / overflowed fp32 worker: one source (histogram counts / full norm sweep);
        // fp32 normal case: threshold-free bins from sweep 2 plus the candidate keys.
        double E = 0.0;
        if (is_bf16 || cand_overflow[m]) {
            for (int c = 0; c < n_band; ++c) E += band_partial[((int64_t)m * norm_ctas + c) * kMaxLevels + l];
        } else {
            for (int c = 0; c < n_sum; ++c) E += sum_partial[((int64_t)m * sum_ctas + c) * kMaxLevels + l];
            // candidate keys of the two boundary bins that meet this interval: exact integer sums of mant^2
            for (int side = 0; side < 2; ++side) {
                const unsigned long long* S = cand_S + ((int64_t)m * kMaxLevels + l) * 4 + side * 2;
                const int j = side ? l : l - 1;  // the threshold whose bin fixes the exponent
                if ((S[0] | S[1]) && j >= 0 && j < L - 1) {
                    const int e = (int)(q[j].T >> 23);
                    const unsigned __int128 tot = ((unsigned __int128)S[1] << 24) + S[0];
                    const double td = (double)(unsigned long long)(tot >> 64) * 0x1.0p64 + (double)(unsigned long long)tot;
                    E += ldexp(td, 2 * ((e ? e : 1) - 150));
                }
            }
        }
        const int64_t lo = l ? k[l - 1] : 0, hi = k[l];
        for (int j = 0; j < L - 1; ++j) {
            if (!sh_first[j]) continue;  // trivial, or the same threshold key as an earlier query
            const int64_t c0 = sh_c[j], c1 = c0 + (int64_t)sh_n[j];
            const int64_t ov = min(c1, hi) - max(c0, lo);
            if (ov > 0) {
                const uint32_t bits = is_bf16 ? (sh_T[j] << 16) : sh_T[j];
                const double x = (double)__uint_as_float(bits);
                E = fma((double)ov, x * x, E);
            }
        }
        sh_delta[l] = sqrt(E);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double p_sel;
        int level;
        if (adaptive) {
            double s = 0.0;
            for (int i = 0; i < L; ++i) s += sh_delta[i];
            for (int i = 0; i < L; ++i) {
                sh_p[i] = (s > 0.0) ? sh_delta[i] / s : (i == 0 ? 1.0 : 0.0);
                p_all[m * kMaxLevels + i] = sh_p[i];
                delta_all[m * kMaxLevels + i] = sh_delta[i];
            }
            const double u = counter_uniform(seed, step, (uint64_t)m);
            u_dev[m] = u;
            level = draw_level(sh_p, L, u);
            p_sel = sh_p[level];
        } else {
            level = emit[m].level;  // drawn before the sweeps
            p_sel = p_all[m * kMaxLevels + level];
        }
        if (want_emit)
            fill_emit(m, level, p_sel, q, k, L, d, emit, out_count, out_level, out_p_sel, capacity, status, worker_err);
    }
}

__global__ void copy_probs_kernel(const double* p_all, const double* delta_all, const double* p_fixed, int M, int L,
                                  double* p_out, double* delta_out, const int* worker_err) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * L) return;
    const int m = i / L, l = i % L;
    const bool bad = worker_err[m] != 0;
    if (p_out) p_out[i] = p_fixed ? p_fixed[l] : (bad ? 0.0 : p_all[m * kMaxLevels + l]);
    if (delta_out) delta_out[i] = bad ? 0.0 : delta_all[m * kMaxLevels + l];
}

// -------------------------------------------------------------------------------------------
// s-Top-k with more levels than kMaxLevels (fixed p): the level is drawn first, and the two ranks that bound its
// segment, s l and min(d, s (l + 1)), are the only queries (Sec. 3.2: the residual is the l-th segment)
// -------------------------------------------------------------------------------------------
__global__ void stopk_draw_kernel(const double* __restrict__ p_big, const double* __restrict__ cdf_big, int64_t L,
                                  int64_t s_len, int64_t d, uint64_t seed, uint64_t step, int M, double* p_all,
                                  double* u_dev, EmitParams* emit, Query* queries) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    const double u = counter_uniform(seed, step, (uint64_t)m);
    u_dev[m] = u;
    int64_t lo = 0, hi = L - 1;  // l* = min{ l : u < cdf_l }; the running sums are nondecreasing and end at 1 > u
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (u < cdf_big[mid]) hi = mid; else lo = mid + 1;
    }
    emit[m].level = (int32_t)lo;
    p_all[m * kMaxLevels] = p_big[lo];
    const int64_t kk[2] = {s_len * lo, min(d, s_len * (lo + 1))};
    for (int j = 0; j < 2; ++j) {
        Query q = {};
        q.k = (uint32_t)kk[j];
        q.slot = kNoSlot;
        q.trivial = (kk[j] <= 0) ? 1u : (kk[j] >= d ? 2u : 0u);
        if (q.trivial == 1u) {
            q.T = kKeyNone;
        } else if (q.trivial == 2u) {
            q.T = 0u;
            q.r = 0xFFFFFFFFu;
        }
        queries[m * kMaxQueries + j] = q;
    }
}

__global__ void stopk_params_kernel(const Query* queries, int64_t s_len, int64_t d, const double* p_all, EmitParams* emit,
                                    int64_t* out_count, int32_t* out_level, double* out_p_sel, int64_t capacity,
                                    int* status, int* worker_err, int M) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    if (worker_err[m]) {
        fail_worker(m, emit, out_count, out_level, out_p_sel);
        return;
    }
    const int32_t level = emit[m].level;
    // the segment as the middle band of the three-level schedule (s l, min(d, s (l + 1)), d)
    const int64_t k3[3] = {s_len * level, min(d, s_len * ((int64_t)level + 1)), d};
    fill_emit(m, 1, p_all[m * kMaxLevels], queries + m * kMaxQueries, k3, 3, d, emit, out_count, out_level, out_p_sel,
              capacity, status, worker_err);
    if (emit[m].enabled) {
        emit[m].level = level;
        out_level[m] = level;
    }
}

// Everything a selection accumulates into, cleared by one launch: the three histograms, the tile maxima, the
// candidate counters and sums (zero), and the digit-2 slot map ("no slot").
struct ResetList {
    uint32_t* ptr[8];
    uint32_t words[8];
    uint32_t value[8];
    int n;
};

__global__ void reset_state_kernel(ResetList r) {
    for (int a = 0; a < r.n; ++a) {
        uint32_t* p = r.ptr[a];
        const uint32_t n4 = r.words[a] / 4, v = r.value[a];
        for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x)
            reinterpret_cast<uint4*>(p)[i] = make_uint4(v, v, v, v);
        for (uint32_t i = n4 * 4 + blockIdx.x * blockDim.x + threadIdx.x; i < r.words[a]; i += gridDim.x * blockDim.x) p[i] = v;
    }
}

int blocks_per_worker(const Workspace& ws, int64_t d, int vec, int threads, int M, int waves) {
    const int64_t nvec = (d + vec - 1) / vec;
    const int64_t by_work = (nvec + (int64_t)threads * 4 - 1) / ((int64_t)threads * 4);
    int64_t by_sm = ((int64_t)ws.sm_count * waves) / M;  // rounded down: one block too many per worker costs a whole extra wave
    if (by_sm < 1) by_sm = 1;
    int64_t nb = by_work < by_sm ? by_work : by_sm;
    return (int)(nb < 1 ? 1 : nb);
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
void launch_init_queries_adaptive(Workspace& ws, int M, int L, int64_t d, cudaStream_t s) {
    if (L > 1) {
        LaunchScope t(ws, K_INIT_QUERIES, s);
        init_queries_kernel<<<M, kMaxQueries, 0, s>>>(ws.queries, ws.k_dev, L, d, ws.emit, 0, nullptr, nullptr);
    }
}

void launch_draw_fixed(Workspace& ws, int M, int L, int64_t d, uint64_t seed, uint64_t step, bool brackets,
                       cudaStream_t s) {
    {
        LaunchScope t(ws, K_DRAW_FIXED, s);
        draw_fixed_kernel<<<(M + 127) / 128, 128, 0, s>>>(ws.p_fixed, L, seed, step, ws.p_all, ws.u_dev, ws.emit, M);
    }
    if (L > 1) {
        LaunchScope t(ws, K_INIT_QUERIES, s);
        init_queries_kernel<<<M, kMaxQueries, 0, s>>>(ws.queries, ws.k_dev, L, d, ws.emit, 1, ws.prev_bin,
                                                      brackets ? ws.bracket : nullptr);
    }
}

void launch_uniforms(Workspace& ws, int M, uint64_t seed, uint64_t step, cudaStream_t s) {
    LaunchScope t(ws, K_UNIFORMS, s);
    uniforms_kernel<<<(M + 127) / 128, 128, 0, s>>>(ws.u_dev, M, seed, step);
}

// One launch instead of nine memsets, before the first sweep.
void launch_reset_selection(Workspace& ws, int dtype, int64_t d, int M, cudaStream_t s) {
    const int tpw = emit_tiles_per_worker(d, dtype);
    ResetList r = {};
    auto add = [&](void* p, size_t bytes, uint32_t value) {
        r.ptr[r.n] = static_cast<uint32_t*>(p);
        r.words[r.n] = (uint32_t)(bytes / 4);
        r.value[r.n] = value;
        ++r.n;
    };
    add(ws.hist1, (size_t)M * kBins1 * sizeof(uint32_t), 0u);
    add(ws.tile_max, (size_t)M * tpw * kEmitGroups * sizeof(uint32_t), 0u);
    if (dtype == MLMC_F32) {
        add(ws.cand_count, sizeof(uint32_t) * M, 0u);
        add(ws.cand_overflow, sizeof(int) * M, 0u);
        add(ws.hist2, (size_t)M * kMaxQueries * kBins23 * sizeof(uint32_t), 0u);
        add(ws.map2, (size_t)M * kMaxQueries * kBins23, 0xFFFFFFFFu);
        add(ws.hist3, (size_t)M * kMaxQueries * kBins23 * sizeof(uint32_t), 0u);
        add(ws.cand_S, (size_t)M * kMaxLevels * 4 * sizeof(unsigned long long), 0u);
    }
    LaunchScope t(ws, K_RESET, s);
    reset_state_kernel<<<ws.sm_count * 2, 512, 0, s>>>(r);
}

void launch_hist1(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, bool brackets, cudaStream_t s) {
    const int tpw = emit_tiles_per_worker(d, dtype);
    const size_t smem = kBins1 * sizeof(uint32_t);
    LaunchScope t(ws, K_HIST1, s);
    if (dtype == MLMC_BF16) {
        const int nb = blocks_per_worker(ws, d, 8, kHistThreads, M, 2);
        hist1_kernel<bf16_t, false><<<dim3(nb, M), kHistThreads, smem, s>>>(
            static_cast<const bf16_t*>(g), d, ld, ws.hist1, ws.tile_max, tpw, ws.status, ws.worker_err, nullptr, nullptr, 0,
            nullptr, nullptr);
    } else {
        const int nb = blocks_per_worker(ws, d, 4, kHistThreads, M, 2);
        if (brackets)
            hist1_kernel<float, true><<<dim3(nb, M), kHistThreads, smem + (kHistThreads / 32) * (kWarpStage + 1) * sizeof(uint32_t), s>>>(
                static_cast<const float*>(g), d, ld, ws.hist1, ws.tile_max, tpw, ws.status, ws.worker_err, ws.bracket,
                ws.cand_keys, ws.cand_cap, ws.cand_count, ws.cand_overflow);
        else
            hist1_kernel<float, false><<<dim3(nb, M), kHistThreads, smem, s>>>(
                static_cast<const float*>(g), d, ld, ws.hist1, ws.tile_max, tpw, ws.status, ws.worker_err, nullptr, nullptr,
                0, nullptr, nullptr);
    }
}

void launch_resolve1(Workspace& ws, int dtype, int M, int L, bool brackets, cudaStream_t s) {
    LaunchScope t(ws, K_RESOLVE1, s);
    resolve1_kernel<<<M, kResolveThreads, 0, s>>>(ws.hist1, ws.queries, ws.table1, ws.cand_floor, L - 1,
                                                  dtype == MLMC_BF16, ws.worker_err, ws.emit,
                                                  brackets ? ws.bracket : nullptr, ws.bracket_hit, ws.prev_bin,
                                                  ws.bracket_stats, ws.cand_count, ws.cand_overflow);
}

static int cand_blocks(const Workspace& ws, int M) {
    int nb = (ws.sm_count * 2) / M;
    return nb < 1 ? 1 : nb;
}

static size_t s2_smem(int L, bool sums) {
    return kBins1 + (size_t)kStage * 4 + (sums ? (size_t)L * kS2Threads * sizeof(double) : 0);
}

// Sweep 2: energies of the threshold-free bins (adaptive only) and the candidate keys of the boundary bins.
void launch_sums_candidates(Workspace& ws, const void* g, int64_t d, int M, int64_t ld, int L, bool sums,
                            bool brackets, cudaStream_t s) {
    int nb = blocks_per_worker(ws, d, 4, kS2Threads, M, sums ? 2 : 8);  // without the accumulators four blocks fit an SM
    if (nb > ws.sum_ctas) nb = ws.sum_ctas;
    ws.cur_sum_ctas = nb;
    const size_t smem = s2_smem(L, sums);
    LaunchScope t(ws, K_SUMS_CAND, s);
    if (sums)
        sums_candidates_kernel<true><<<dim3(nb, M), kS2Threads, smem, s>>>(
            static_cast<const float*>(g), d, ld, ws.table1, L, ws.sum_partial, ws.sum_ctas, ws.cand_keys,
            ws.cand_cap, ws.cand_count, ws.cand_overflow, ws.worker_err, ws.tile_max,
            emit_tiles_per_worker(d, MLMC_F32), ws.cand_floor, nullptr);
    else
        sums_candidates_kernel<false><<<dim3(nb, M), kS2Threads, smem, s>>>(
            static_cast<const float*>(g), d, ld, ws.table1, L, ws.sum_partial, ws.sum_ctas, ws.cand_keys,
            ws.cand_cap, ws.cand_count, ws.cand_overflow, ws.worker_err, ws.tile_max,
            emit_tiles_per_worker(d, MLMC_F32), ws.cand_floor, brackets ? ws.bracket_hit : nullptr);
}

// Digit pass 2 or 3: over the candidate keys, and (early exit unless the buffer overflowed) over the full row.
void launch_digit_pass(Workspace& ws, const void* g, int64_t d, int M, int64_t ld, int pass, cudaStream_t s) {
    const size_t smem = kMaxQueries * kBins23 * sizeof(uint32_t) + kBins1 + kMaxQueries * kBins23;
    const int nb_full = blocks_per_worker(ws, d, 4, kSweepThreads, M, 2);  // fall-back sweeps: a small grid, since they normally exit at once
    const int nb_cand = cand_blocks(ws, M);
    LaunchScope t(ws, pass == 2 ? K_CAND2 : K_CAND3, s);
    if (pass == 2)
        digit_pass_kernel<2><<<dim3(nb_cand + nb_full, M), kSweepThreads, smem, s>>>(
            nb_cand, static_cast<const float*>(g), d, ld, ws.cand_keys, ws.cand_cap, ws.cand_count, ws.cand_overflow,
            ws.table1, ws.map2, ws.hist2, ws.worker_err);
    else
        digit_pass_kernel<3><<<dim3(nb_cand + nb_full, M), kSweepThreads, smem, s>>>(
            nb_cand, static_cast<const float*>(g), d, ld, ws.cand_keys, ws.cand_cap, ws.cand_count, ws.cand_overflow,
            ws.table1, ws.map2, ws.hist3, ws.worker_err);
}

void launch_resolve23(Workspace& ws, int M, int L, int pass, cudaStream_t s) {
    LaunchScope t(ws, pass == 2 ? K_RESOLVE2 : K_RESOLVE3, s);
    if (pass == 2)
        resolve23_kernel<2><<<M, kResolveThreads, 0, s>>>(ws.hist2, ws.queries, ws.map2, L - 1, ws.worker_err);
    else
        resolve23_kernel<3><<<M, kResolveThreads, 0, s>>>(ws.hist3, ws.queries, ws.map2, L - 1, ws.worker_err);
}

// Band energies of the boundary bins from the candidate keys, and the full-sweep fallback.
void launch_band_norms_fp32(Workspace& ws, const void* g, int64_t d, int M, int64_t ld, int L, cudaStream_t s) {
    {
        const int nb = 3 * cand_blocks(ws, M);
        LaunchScope t(ws, K_CAND_SUMS, s);
        cand_sums_kernel<<<dim3(nb, M), kCandSumThreads, (size_t)L * 4 * kCandSumThreads * sizeof(unsigned long long), s>>>(
            ws.cand_keys, ws.cand_cap, ws.cand_count, ws.cand_overflow, ws.queries, L, ws.cand_S, ws.worker_err);
    }
    int nb = blocks_per_worker(ws, d, 4, kSweepThreads, M, 2);
    if (nb > ws.norm_ctas) nb = ws.norm_ctas;
    ws.cur_norm_ctas = nb;
    const size_t smem = (size_t)L * kSweepThreads * sizeof(double);
    LaunchScope t(ws, K_NORM_SWEEP, s);
    norm_sweep_kernel<<<dim3(nb, M), kSweepThreads, smem, s>>>(static_cast<const float*>(g), d, ld, ws.queries, L,
                                                               ws.band_partial, ws.norm_ctas, ws.worker_err,
                                                               ws.cand_overflow);
}

void launch_norm_from_hist_bf16(Workspace& ws, int M, int L, cudaStream_t s) {
    ws.cur_norm_ctas = kNormParts;
    LaunchScope t(ws, K_NORM_HIST, s);
    norm_from_hist_bf16_kernel<<<dim3(kNormParts, M), kNormThreads, 0, s>>>(ws.hist1, ws.queries, L, ws.band_partial,
                                                                            ws.norm_ctas, ws.worker_err);
}

void launch_probs_draw(Workspace& ws, int dtype, int M, int L, int64_t d, bool adaptive, bool want_emit,
                       uint64_t seed, uint64_t step, const mlmc_topk_msgs* out, cudaStream_t s) {
    LaunchScope t(ws, K_PROBS_DRAW, s);
    probs_draw_kernel<<<M, kMaxLevels, 0, s>>>(
        ws.queries, ws.k_dev, L, d, dtype == MLMC_BF16, ws.band_partial, ws.norm_ctas, ws.cur_norm_ctas,
        ws.sum_partial, ws.sum_ctas, ws.cur_sum_ctas, ws.cand_S,
        ws.cand_overflow, adaptive ? 1 : 0, seed, step, ws.p_all, ws.delta_all, ws.u_dev, ws.emit,
        out ? out->count : nullptr, out ? out->level : nullptr, out ? out->p_sel : nullptr, out ? out->capacity : 0,
        ws.status, ws.worker_err, want_emit ? 1 : 0);
}

void launch_copy_probs(Workspace& ws, int M, int L, const double* p_fixed, double* p_out, double* delta_out,
                       cudaStream_t s) {
    LaunchScope t(ws, K_COPY_PROBS, s);
    copy_probs_kernel<<<(M * L + 127) / 128, 128, 0, s>>>(ws.p_all, ws.delta_all, p_fixed, M, L, p_out, delta_out,
                                                          ws.worker_err);
}

void launch_stopk_draw(Workspace& ws, int M, int64_t L, int64_t s_len, int64_t d, uint64_t seed, uint64_t step,
                       cudaStream_t s) {
    LaunchScope t(ws, K_STOPK_DRAW, s);
    stopk_draw_kernel<<<(M + 127) / 128, 128, 0, s>>>(ws.p_big, ws.cdf_big, L, s_len, d, seed, step, M, ws.p_all, ws.u_dev,
                                                      ws.emit, ws.queries);
}

void launch_stopk_params(Workspace& ws, int M, int64_t s_len, int64_t d, const mlmc_topk_msgs* out, cudaStream_t s) {
    LaunchScope t(ws, K_STOPK_PARAMS, s);
    stopk_params_kernel<<<(M + 127) / 128, 128, 0, s>>>(ws.queries, s_len, d, ws.p_all, ws.emit, out->count, out->level,
                                                        out->p_sel, out->capacity, ws.status, ws.worker_err, M);
}

int configure_select_kernels() {
    cudaError_t e = cudaFuncSetAttribute(hist1_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kBins1 * sizeof(uint32_t)));
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    e = cudaFuncSetAttribute(hist1_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(kBins1 * sizeof(uint32_t) + (kHistThreads / 32) * (kWarpStage + 1) * sizeof(uint32_t)));
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    e = cudaFuncSetAttribute(hist1_kernel<bf16_t, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(kBins1 * sizeof(uint32_t)));
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    const int smem_masked = kMaxQueries * kBins23 * sizeof(uint32_t) + kBins1 + kMaxQueries * kBins23;
    e = cudaFuncSetAttribute(digit_pass_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_masked);
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    e = cudaFuncSetAttribute(digit_pass_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_masked);
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    e = cudaFuncSetAttribute(norm_sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(kMaxLevels * kSweepThreads * sizeof(double)));
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    const int smem_s2 = (int)s2_smem(kMaxLevels, true);
    e = cudaFuncSetAttribute(sums_candidates_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_s2);
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    e = cudaFuncSetAttribute(sums_candidates_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_s2);
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    e = cudaFuncSetAttribute(cand_sums_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(kMaxLevels * 4 * kCandSumThreads * sizeof(unsigned long long)));
    if (e != cudaSuccess) return MLMC_ERR_CUDA;
    return MLMC_OK;
}

}  // namespace mlmc
