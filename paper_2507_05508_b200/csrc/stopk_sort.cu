// s-Top-k with adaptive probabilities and more segments than kMaxLevels (Sec. 2.2 "s-segmented Top-k", App. D,
// Lemma 3.4: p^l proportional to the norm of segment l of the sorted vector).
//
// With up to 32 levels the thresholds of all level boundaries come from one histogram sweep.  With hundreds of
// segments (the paper's Adaptive MLMC-Top-k runs use segments of 1 % to 50 % of the vector, App. D / Sec. 5) nearly
// every histogram bin holds a boundary, so this path sorts the magnitude keys of a row instead (least-significant-
// digit radix sort, 8 bits per pass, keys only: equal keys have equal energy, so the order among them is
// irrelevant here) and reads everything off the sorted row: the norm of every segment, and, for the drawn segment,
// its two thresholds with their counts.  The emission of the band then runs as for every other Top-k message.
// One row is sorted at a time, in two key buffers of d words each that the context allocates at first use.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kSortThreads = 256;
constexpr int kSortItems = 128;                             // keys per thread
constexpr int kSortTile = kSortThreads * kSortItems;        // keys per block: every warp owns 4096 consecutive keys
constexpr int kSortWarps = kSortThreads / 32;
constexpr uint32_t kSortFlip = 0x7FFFFFFFu;                 // sort key = flip - magnitude key: ascending sort, descending magnitude

template <typename T>
__global__ void __launch_bounds__(kSortThreads)
sort_keys_kernel(const T* __restrict__ row, int64_t d, uint32_t* __restrict__ out) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
        uint32_t bits;
        if constexpr (sizeof(T) == 4)
            bits = reinterpret_cast<const uint32_t*>(row)[i];
        else
            bits = reinterpret_cast<const uint16_t*>(row)[i];
        out[i] = kSortFlip - ElemTraits<T>::key(bits);
    }
}

// Digit counts of one warp's 4096 consecutive keys, in its row of the shared-memory table.  The keys are taken 32
// at a time in order; lanes with the same digit find each other by ballots, the lowest of them adds their number.
constexpr int kSortAhead = 8;  // keys per lane requested together

// The lanes of the warp whose key has the same 8-bit digit as this lane's (live lanes only): one ballot per digit
// bit, a constant cost whatever the number of distinct digits.
__device__ __forceinline__ uint32_t same_digit_lanes(uint32_t digit, bool live) {
    uint32_t peers = __ballot_sync(0xFFFFFFFFu, live);
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const bool bit = (digit >> b) & 1u;
        const uint32_t mk = __ballot_sync(0xFFFFFFFFu, bit);
        peers &= bit ? mk : ~mk;
    }
    return peers;
}

__device__ __forceinline__ void warp_digit_counts(const uint32_t* __restrict__ in, int64_t n, int64_t w0, int shift,
                                                  uint32_t* my_hist, int lane) {
    for (int st0 = 0; st0 < kSortItems; st0 += kSortAhead) {
        if (w0 + (int64_t)st0 * 32 >= n) break;  // warp-uniform
        uint32_t digit[kSortAhead];
#pragma unroll
        for (int j = 0; j < kSortAhead; ++j) {
            const int64_t i = w0 + (int64_t)(st0 + j) * 32 + lane;
            digit[j] = (i < n) ? ((in[i] >> shift) & 0xFFu) : 256u;  // 256: past the end
        }
#pragma unroll
        for (int j = 0; j < kSortAhead; ++j) {
            const uint32_t peers = same_digit_lanes(digit[j], digit[j] < 256u);
            if (digit[j] < 256u && (peers & ((1u << lane) - 1u)) == 0u) my_hist[digit[j]] += __popc(peers);
            __syncwarp();
        }
    }
}

// block_hist[digit][block] = keys of the block's tile with that digit.
__global__ void __launch_bounds__(kSortThreads)
sort_count_kernel(const uint32_t* __restrict__ in, int64_t n, int shift, uint32_t* __restrict__ block_hist, int nblocks) {
    __shared__ uint32_t sh_hist[kSortWarps][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kSortWarps * 256; i += kSortThreads) (&sh_hist[0][0])[i] = 0u;
    __syncthreads();
    warp_digit_counts(in, n, (int64_t)blockIdx.x * kSortTile + (int64_t)warp * (kSortItems * 32), shift, sh_hist[warp], lane);
    __syncthreads();
    uint32_t tot = 0;
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) tot += sh_hist[w][threadIdx.x];
    block_hist[(int64_t)threadIdx.x * nblocks + blockIdx.x] = tot;
}

// Exclusive scan of the digit-major table in place (one block): every warp owns a contiguous range (a multiple of
// 32 entries, read as coalesced rows), adds it up, and after one barrier scans it row by row from the total of the
// warps before it.
__global__ void __launch_bounds__(1024)
sort_scan_kernel(uint32_t* __restrict__ table, int64_t total) {
    __shared__ uint32_t sh_warp[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t rows = (total + 1023) / 1024;  // rows of 32 entries per warp
    const int64_t t0 = (int64_t)warp * rows * 32;
    uint32_t sum = 0;
#pragma unroll 4
    for (int64_t r = 0; r < rows; ++r) {
        const int64_t i = t0 + r * 32 + lane;
        if (i < total) sum += table[i];
    }
    sum = __reduce_add_sync(0xFFFFFFFFu, sum);
    if (lane == 0) sh_warp[warp] = sum;
    __syncthreads();
    uint32_t carry = 0;
    for (int w = 0; w < warp; ++w) carry += sh_warp[w];
    for (int64_t r = 0; r < rows; ++r) {
        const int64_t i = t0 + r * 32 + lane;
        if (t0 + r * 32 >= total) break;  // warp-uniform
        const uint32_t x = (i < total) ? table[i] : 0u;
        uint32_t incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += y;
        }
        if (i < total) table[i] = carry + incl - x;
        carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
}

// Stable scatter of one pass: a key goes to (start of its digit for this block) + (keys with that digit in the warps
// before) + (its rank among the warp's keys with that digit, in order).
__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const uint32_t* __restrict__ in, uint32_t* __restrict__ out, int64_t n, int shift,
                    const uint32_t* __restrict__ block_base, int nblocks) {
    __shared__ uint32_t sh_hist[kSortWarps][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kSortWarps * 256; i += kSortThreads) (&sh_hist[0][0])[i] = 0u;
    __syncthreads();
    const int64_t w0 = (int64_t)blockIdx.x * kSortTile + (int64_t)warp * (kSortItems * 32);
    warp_digit_counts(in, n, w0, shift, sh_hist[warp], lane);
    __syncthreads();
    {  // per digit: where each warp's keys start
        uint32_t run = block_base[(int64_t)threadIdx.x * nblocks + blockIdx.x];
#pragma unroll
        for (int w = 0; w < kSortWarps; ++w) {
            const uint32_t c = sh_hist[w][threadIdx.x];
            sh_hist[w][threadIdx.x] = run;
            run += c;
        }
    }
    __syncthreads();
    uint32_t* my_base = sh_hist[warp];
    for (int st0 = 0; st0 < kSortItems; st0 += kSortAhead) {
        if (w0 + (int64_t)st0 * 32 >= n) break;  // warp-uniform
        uint32_t key[kSortAhead];
        bool live[kSortAhead];
#pragma unroll
        for (int j = 0; j < kSortAhead; ++j) {
            const int64_t i = w0 + (int64_t)(st0 + j) * 32 + lane;
            live[j] = i < n;
            key[j] = live[j] ? in[i] : 0u;
        }
#pragma unroll
        for (int j = 0; j < kSortAhead; ++j) {
            const uint32_t digit = (key[j] >> shift) & 0xFFu;
            const uint32_t peers = same_digit_lanes(digit, live[j]);
            const int leader = live[j] ? __ffs(peers) - 1 : lane;
            uint32_t base = 0;
            if (live[j] && lane == leader) {
                base = my_base[digit];
                my_base[digit] = base + __popc(peers);
            }
            base = __shfl_sync(0xFFFFFFFFu, base, leader);
            if (live[j]) out[base + __popc(peers & ((1u << lane) - 1u))] = key[j];
            __syncwarp();
        }
    }
}

// Norm of every segment of the sorted row in fp64, in a fixed order (reproducible): a group of G lanes (one warp,
// or a whole block for long segments) strides over the segment, then a shuffle tree per warp and the warp sums in
// warp order.
template <bool BLOCK>
__global__ void __launch_bounds__(256)
segment_norms_kernel(const uint32_t* __restrict__ sorted, int64_t d, int64_t s_len, int64_t L, int is_bf16,
                     double* __restrict__ delta) {
    __shared__ double sh_w[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t seg = BLOCK ? (int64_t)blockIdx.x : (int64_t)blockIdx.x * 8 + warp;
    if (seg >= L) return;  // block-uniform when BLOCK
    const int64_t lo = seg * s_len, hi = min(d, lo + s_len);
    double acc = 0.0;
    for (int64_t i = lo + (BLOCK ? (int)threadIdx.x : lane); i < hi; i += BLOCK ? 256 : 32) {
        const uint32_t key = kSortFlip - sorted[i];
        const double x = (double)__uint_as_float(is_bf16 ? (key << 16) : key);
        acc = fma(x, x, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (!BLOCK) {
        if (lane == 0) delta[seg] = sqrt(acc);
        return;
    }
    if (lane == 0) sh_w[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int w = 0; w < 8; ++w) tot += sh_w[w];
        delta[seg] = sqrt(tot);
    }
}

// p_l = Delta_l / sum Delta (Lemma 3.4), the level draw by the running sums of p, and the two thresholds of the drawn
// segment read off the sorted row.  One block for the one worker in hand.
__global__ void __launch_bounds__(1024)
stopk_sorted_draw_kernel(const uint32_t* __restrict__ sorted, const double* __restrict__ delta, int64_t d,
                         int64_t s_len, int64_t L, int m, uint64_t seed, uint64_t step, double* p_all, double* u_dev,
                         EmitParams* emit, Query* queries) {
    __shared__ double sh_sum[1024];
    __shared__ long long sh_last[1024];
    __shared__ long long sh_level;
    const int t = threadIdx.x;
    const int64_t per = (L + 1023) / 1024;
    const int64_t l0 = min((int64_t)t * per, L), l1 = min(l0 + per, L);
    double part = 0.0;
    long long last = -1;  // last level of the chunk with a positive norm
    for (int64_t l = l0; l < l1; ++l) {
        part += delta[l];
        if (delta[l] > 0.0) last = l;
    }
    sh_sum[t] = part;
    sh_last[t] = last;
    if (t == 0) sh_level = -1;
    __syncthreads();
    double total = 0.0, before = 0.0, end = 0.0;
    long long j_last = -1;
    for (int i = 0; i < 1024; ++i) {  // fixed order, the same in every thread: the chunks tile [0, total] exactly
        if (i == t) before = total;
        total += sh_sum[i];
        if (i == t) end = total;
        j_last = max(j_last, sh_last[i]);
    }
    const double u = counter_uniform(seed, step, (uint64_t)m);
    // l* = min{ l : u < cdf_l } with cdf_l = (Delta_0 + ... + Delta_l) / total.  Exactly one chunk has
    // before / total <= u < end / total; its thread walks it.  (A level past the last positive norm cannot be drawn:
    // the running sum does not grow there.)
    if (total > 0.0 && before / total <= u && u < end / total) {
        double c = before;
        long long found = last;  // if rounding hides the crossing: the chunk's last level with a positive norm
        for (int64_t l = l0; l < l1; ++l) {
            c += delta[l];
            if (u < c / total) {
                found = l;
                break;
            }
        }
        sh_level = found;
    }
    __syncthreads();
    if (t != 0) return;
    int64_t level = (total > 0.0) ? (int64_t)sh_level : 0;
    if (level < 0) level = (j_last >= 0) ? (int64_t)j_last : 0;
    const double p_sel = (total > 0.0) ? delta[level] / total : 1.0;
    u_dev[m] = u;
    p_all[m * kMaxLevels] = p_sel;
    emit[m].level = (int32_t)level;
    // the two ranks that bound the segment, and their thresholds from the sorted row (descending magnitude):
    // T = key of rank k, c = keys above it, n = keys equal to it
    const int64_t kk[2] = {s_len * level, min(d, s_len * (level + 1))};
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
        } else {
            const uint32_t sk = sorted[kk[j] - 1];
            int64_t lo = 0, hi = kk[j] - 1;  // first position holding sk
            while (lo < hi) {
                const int64_t mid = (lo + hi) >> 1;
                if (sorted[mid] < sk) lo = mid + 1; else hi = mid;
            }
            int64_t lo2 = kk[j] - 1, hi2 = d;  // first position past sk
            while (lo2 < hi2) {
                const int64_t mid = (lo2 + hi2) >> 1;
                if (sorted[mid] <= sk) lo2 = mid + 1; else hi2 = mid;
            }
            q.T = kSortFlip - sk;
            q.c = (uint32_t)lo;
            q.n = (uint32_t)(lo2 - lo);
            q.r = (uint32_t)(kk[j] - lo);
        }
        queries[m * kMaxQueries + j] = q;
    }
}

}  // namespace

size_t stopk_sort_scratch_words(int64_t d_max) {
    const int64_t nblocks = (d_max + kSortTile - 1) / kSortTile;
    return (size_t)(2 * d_max + 256 * nblocks);
}

// Sorts row m, writes its segment norms to ws.delta_big, draws its level and fills its two queries.
void launch_stopk_sorted_worker(Workspace& ws, const void* g, int dtype, int64_t d, int m, int64_t ld, int64_t s_len,
                                int64_t L, uint64_t seed, uint64_t step, cudaStream_t s) {
    uint32_t* buf_a = ws.sort_scratch;
    uint32_t* buf_b = buf_a + ws.d_max;
    uint32_t* table = buf_b + ws.d_max;
    const int nblocks = (int)((d + kSortTile - 1) / kSortTile);
    const int grid_keys = (int)(((d + kSortThreads - 1) / kSortThreads < (int64_t)ws.sm_count * 16)
                                    ? (d + kSortThreads - 1) / kSortThreads : (int64_t)ws.sm_count * 16);
    {
        LaunchScope t(ws, K_SORT_KEYS, s);
        if (dtype == MLMC_BF16)
            sort_keys_kernel<bf16_t><<<grid_keys, kSortThreads, 0, s>>>(static_cast<const bf16_t*>(g) + (int64_t)m * ld, d, buf_a);
        else
            sort_keys_kernel<float><<<grid_keys, kSortThreads, 0, s>>>(static_cast<const float*>(g) + (int64_t)m * ld, d, buf_a);
    }
    const int passes = (dtype == MLMC_BF16) ? 2 : 4;  // 15-bit and 31-bit keys
    uint32_t* src = buf_a;
    uint32_t* dst = buf_b;
    for (int p = 0; p < passes; ++p) {
        {
            LaunchScope t(ws, K_SORT_PASS, s);
            sort_count_kernel<<<nblocks, kSortThreads, 0, s>>>(src, d, 8 * p, table, nblocks);
        }
        {
            LaunchScope t(ws, K_SORT_PASS, s);
            sort_scan_kernel<<<1, 1024, 0, s>>>(table, (int64_t)256 * nblocks);
        }
        {
            LaunchScope t(ws, K_SORT_PASS, s);
            sort_scatter_kernel<<<nblocks, kSortThreads, 0, s>>>(src, dst, d, 8 * p, table, nblocks);
        }
        uint32_t* tmp = src;
        src = dst;
        dst = tmp;
    }
    {
        LaunchScope t(ws, K_SEG_NORMS, s);
        if (s_len >= 4096)
            segment_norms_kernel<true><<<(unsigned)L, 256, 0, s>>>(src, d, s_len, L, dtype == MLMC_BF16, ws.cdf_big);
        else
            segment_norms_kernel<false><<<(unsigned)((L + 7) / 8), 256, 0, s>>>(src, d, s_len, L, dtype == MLMC_BF16,
                                                                                ws.cdf_big);
    }
    LaunchScope t(ws, K_STOPK_DRAW, s);
    stopk_sorted_draw_kernel<<<1, 1024, 0, s>>>(src, ws.cdf_big, d, s_len, L, m, seed, step, ws.p_all, ws.u_dev, ws.emit,
                                                ws.queries);
}

}  // namespace mlmc
