// s-Top-k with adaptive probabilities and more segments than kMaxLevels (Sec. 2.2 "s-segmented Top-k", App. D,
// Lemma 3.4: p^l proportional to the norm of segment l of the sorted vector).
//
// With up to 32 levels the thresholds of all level boundaries come from one histogram sweep.  With hundreds of
// segments (the paper's Adaptive MLMC-Top-k runs use segments of 1 % to 50 % of the vector, App. D / Sec. 5) nearly
// every histogram bin holds a boundary, so this path sorts the magnitude keys of a row instead (least-significant-
// digit radix sort, 8 bits per pass, keys only: equal keys have equal energy, so the order among them is
// irrelevant here) and reads everything off the sorted row: the norm of every segment, and, for the drawn segment,
// its two thresholds with their counts.  The emission of the band then runs as for every other Top-k message.
// As many rows are sorted together as fit in a fixed budget of scratch memory (two key buffers of d words per row,
// the digit tables and the norms), which the context allocates at first use.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kSortThreads = 512;
constexpr int kSortItems = 16;                              // keys per thread
constexpr int kSortTile = kSortThreads * kSortItems;        // keys per block
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kWarpKeys = kSortItems * 32;                  // every warp owns this many consecutive keys of the tile
constexpr uint32_t kSortFlip = 0x7FFFFFFFu;                 // sort key = flip - magnitude key: ascending sort, descending magnitude
constexpr int kNormChunk = 4096;                            // keys per block of the segment norms
constexpr size_t kSortScratchBudget = size_t(1) << 30;      // rows are sorted together while their buffers fit in this

// What a pass reads: the sort keys of the pass before, or (first pass) the gradient row itself.
enum { SRC_KEYS = 0, SRC_F32 = 1, SRC_BF16 = 2 };

template <int SRC>
__device__ __forceinline__ const void* sort_row(const void* base, int64_t stride, int row) {
    if constexpr (SRC == SRC_BF16)
        return static_cast<const uint16_t*>(base) + (int64_t)row * stride;
    else
        return static_cast<const uint32_t*>(base) + (int64_t)row * stride;
}

template <int SRC>
__device__ __forceinline__ uint32_t load_sort_key(const void* row, int64_t i) {
    if constexpr (SRC == SRC_KEYS)
        return static_cast<const uint32_t*>(row)[i];
    else if constexpr (SRC == SRC_F32)
        return kSortFlip - ElemTraits<float>::key(static_cast<const uint32_t*>(row)[i]);
    else
        return kSortFlip - ElemTraits<bf16_t>::key(static_cast<const uint16_t*>(row)[i]);
}

// table[row][digit][block] = keys of the block's tile with that digit.
template <int SRC>
__global__ void __launch_bounds__(kSortThreads)
sort_count_kernel(const void* __restrict__ in, int64_t in_stride, int64_t n, int shift, uint32_t* __restrict__ table,
                  int nblocks) {
    __shared__ uint32_t sh_hist[kSortWarps][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kSortWarps * 256; i += kSortThreads) (&sh_hist[0][0])[i] = 0u;
    __syncthreads();
    const void* row = sort_row<SRC>(in, in_stride, blockIdx.y);
    const int64_t w0 = (int64_t)blockIdx.x * kSortTile + (int64_t)warp * kWarpKeys + lane;
    uint32_t key[kSortItems];
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) key[j] = (w0 + j * 32 < n) ? load_sort_key<SRC>(row, w0 + j * 32) : 0u;
#pragma unroll
    for (int j = 0; j < kSortItems; ++j)
        if (w0 + j * 32 < n) atomicAdd(&sh_hist[warp][(key[j] >> shift) & 0xFFu], 1u);
    __syncthreads();
    if (threadIdx.x < 256) {
        uint32_t tot = 0;
#pragma unroll
        for (int w = 0; w < kSortWarps; ++w) tot += sh_hist[w][threadIdx.x];
        table[((int64_t)blockIdx.y * 256 + threadIdx.x) * nblocks + blockIdx.x] = tot;
    }
}

// Exclusive scan, in place, of the block counts of one digit of one row (a block per digit and row); the digit's
// total goes to totals[row][digit].  The scatter adds the totals of the digits below.
__global__ void __launch_bounds__(256)
sort_scan_kernel(uint32_t* __restrict__ tables, uint32_t* __restrict__ totals, int nblocks) {
    __shared__ uint32_t sh_warp[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* entries = tables + ((int64_t)blockIdx.y * 256 + blockIdx.x) * nblocks;
    uint32_t carry = 0;
    for (int i0 = 0; i0 < nblocks; i0 += 256) {  // block-uniform
        const int i = i0 + threadIdx.x;
        const uint32_t x = (i < nblocks) ? entries[i] : 0u;
        uint32_t incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += y;
        }
        if (lane == 31) sh_warp[warp] = incl;
        __syncthreads();
        uint32_t before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const uint32_t v = sh_warp[w];
            if (w < warp) before += v;
            all += v;
        }
        if (i < nblocks) entries[i] = carry + before + incl - x;
        carry += all;
        __syncthreads();
    }
    if (threadIdx.x == 0) totals[blockIdx.y * 256 + blockIdx.x] = carry;
}

constexpr int kScatterSmemWords = kSortTile + 3 * kSortWarps * 256;  // the ordered tile, the warp tables, two mask tables

// Stable scatter of one pass.  The block first orders its tile by digit in shared memory (a key's place: start of
// its digit in the tile + keys with that digit in the warps before + its rank among its warp's keys with that
// digit, in input order), then writes the tile out so that consecutive threads write consecutive keys of a digit's
// run: the runs are contiguous in the output, from the scanned table.
// Ranks within a warp: the warp takes its keys 32 at a time in input order; the lanes of a step that hold the same
// digit meet in a shared-memory word per digit, into which each ORs its lane bit; the lowest of them advances the
// warp's running count of the digit and clears the word (two mask tables alternate, so that a step never meets the
// clearing of the step before).
template <int SRC>
__global__ void __launch_bounds__(kSortThreads, 2)
sort_scatter_kernel(const void* __restrict__ in, int64_t in_stride, uint32_t* __restrict__ out, int64_t out_stride,
                    int64_t n, int shift, const uint32_t* __restrict__ tables, const uint32_t* __restrict__ totals,
                    int nblocks) {
    extern __shared__ __align__(16) uint32_t sh_dyn[];
    uint32_t* sh_key = sh_dyn;                            // [kSortTile]
    uint32_t* sh_hist = sh_dyn + kSortTile;               // [warp][256]
    uint32_t* sh_mask = sh_hist + kSortWarps * 256;       // [2][warp][256]
    __shared__ uint32_t sh_shift[256];  // position in the output - position in the ordered tile, per digit (mod 2^32)
    __shared__ uint32_t sh_wsum[8], sh_gsum[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 3 * kSortWarps * 256; i += kSortThreads) sh_hist[i] = 0u;
    const void* row = sort_row<SRC>(in, in_stride, blockIdx.y);
    const int64_t tile0 = (int64_t)blockIdx.x * kSortTile;
    const int64_t w0 = tile0 + (int64_t)warp * kWarpKeys + lane;
    uint32_t key[kSortItems];
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) key[j] = (w0 + j * 32 < n) ? load_sort_key<SRC>(row, w0 + j * 32) : 0u;
    __syncthreads();
    uint32_t* my_hist = sh_hist + warp * 256;
    uint32_t* my_mask = sh_mask + warp * 256;
    const uint32_t lane_bit = 1u << lane, lanes_below = lane_bit - 1u;
    uint32_t rank2[kSortItems / 2];  // two 16-bit ranks per word
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const bool live = w0 + j * 32 < n;
        const uint32_t digit = (key[j] >> shift) & 0xFFu;
        uint32_t* mask = my_mask + (j & 1) * (kSortWarps * 256) + digit;
        if (live) atomicOr(mask, lane_bit);
        __syncwarp();
        uint32_t peers = 0u, base = 0u;
        if (live) {
            peers = *mask;
            base = my_hist[digit];
        }
        __syncwarp();
        if (live && (peers & lanes_below) == 0u) {
            my_hist[digit] = base + __popc(peers);
            *mask = 0u;
        }
        const uint32_t rank = base + __popc(peers & lanes_below);
        if (j & 1)
            rank2[j >> 1] |= rank << 16;
        else
            rank2[j >> 1] = rank;
    }
    __syncthreads();
    {  // per digit: the tile-local start of every warp's keys, and the shift from the tile order to the output
        uint32_t total = 0, gtotal = 0;  // keys with this digit: in the tile, in the row
        if (threadIdx.x < 256) {
#pragma unroll
            for (int w = 0; w < kSortWarps; ++w) total += sh_hist[w * 256 + threadIdx.x];
            gtotal = totals[blockIdx.y * 256 + threadIdx.x];
        }
        uint32_t incl = total, gincl = gtotal;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            const uint32_t gy = __shfl_up_sync(0xFFFFFFFFu, gincl, o);
            if (lane >= o) {
                incl += y;
                gincl += gy;
            }
        }
        if (threadIdx.x < 256 && lane == 31) {
            sh_wsum[warp] = incl;
            sh_gsum[warp] = gincl;
        }
        __syncthreads();
        if (threadIdx.x < 256) {
            uint32_t start = incl - total, gstart = gincl - gtotal;
            for (int w = 0; w < warp; ++w) {
                start += sh_wsum[w];
                gstart += sh_gsum[w];
            }
            sh_shift[threadIdx.x] =
                gstart + tables[((int64_t)blockIdx.y * 256 + threadIdx.x) * nblocks + blockIdx.x] - start;
            uint32_t run = start;
#pragma unroll
            for (int w = 0; w < kSortWarps; ++w) {
                const uint32_t c = sh_hist[w * 256 + threadIdx.x];
                sh_hist[w * 256 + threadIdx.x] = run;
                run += c;
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        if (w0 + j * 32 < n) {
            const uint32_t rank = (j & 1) ? (rank2[j >> 1] >> 16) : (rank2[j >> 1] & 0xFFFFu);
            sh_key[my_hist[(key[j] >> shift) & 0xFFu] + rank] = key[j];
        }
    }
    __syncthreads();
    const int tile_n = (int)((n - tile0 < (int64_t)kSortTile) ? (n - tile0) : (int64_t)kSortTile);
    uint32_t* out_row = out + (int64_t)blockIdx.y * out_stride;
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const int pos = j * kSortThreads + threadIdx.x;
        if (pos < tile_n) {
            const uint32_t k = sh_key[pos];
            out_row[(uint32_t)pos + sh_shift[(k >> shift) & 0xFFu]] = k;  // mod 2^32
        }
    }
}

__device__ __forceinline__ double key_energy(uint32_t sorted_key, int is_bf16) {
    const uint32_t key = kSortFlip - sorted_key;
    const double x = (double)__uint_as_float(is_bf16 ? (key << 16) : key);
    return x * x;
}

// Norms of the segments of the sorted rows in fp64, in a fixed order (reproducible).  Short segments: one warp per
// segment, the lanes stride over it, a shuffle tree adds them.
__global__ void __launch_bounds__(256)
segment_norms_warp_kernel(const uint32_t* __restrict__ sorted, int64_t stride, int64_t d, int64_t s_len, int64_t L,
                          int is_bf16, double* __restrict__ delta, int64_t delta_stride) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t seg = (int64_t)blockIdx.x * 8 + warp;
    if (seg >= L) return;
    const uint32_t* row = sorted + (int64_t)blockIdx.y * stride;
    const int64_t lo = seg * s_len, hi = min(d, lo + s_len);
    double acc = 0.0;
    for (int64_t i = lo + lane; i < hi; i += 32) acc += key_energy(row[i], is_bf16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) delta[(int64_t)blockIdx.y * delta_stride + seg] = sqrt(acc);
}

// Long segments: a block per chunk of kNormChunk keys of a segment (cps chunks per segment) writes the chunk's energy;
// segment_finish_kernel adds a segment's chunks in order.
__global__ void __launch_bounds__(256)
segment_chunk_energy_kernel(const uint32_t* __restrict__ sorted, int64_t stride, int64_t d, int64_t s_len, int cps,
                            int is_bf16, double* __restrict__ partial, int64_t partial_stride) {
    __shared__ double sh_w[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t seg = (int64_t)blockIdx.x / cps;
    const int chunk = (int)((int64_t)blockIdx.x % cps);
    const uint32_t* row = sorted + (int64_t)blockIdx.y * stride;
    const int64_t seg_hi = min(d, (seg + 1) * s_len);
    const int64_t lo = seg * s_len + (int64_t)chunk * kNormChunk, hi = min(seg_hi, lo + kNormChunk);
    double acc = 0.0;
#pragma unroll 4
    for (int64_t i = lo + threadIdx.x; i < hi; i += 256) acc += key_energy(row[i], is_bf16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) sh_w[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int w = 0; w < 8; ++w) tot += sh_w[w];
        partial[(int64_t)blockIdx.y * partial_stride + blockIdx.x] = tot;
    }
}

__global__ void __launch_bounds__(256)
segment_finish_kernel(const double* __restrict__ partial, int64_t partial_stride, int64_t L, int cps,
                      double* __restrict__ delta, int64_t delta_stride) {
    const int64_t seg = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (seg >= L) return;
    const double* p = partial + (int64_t)blockIdx.y * partial_stride + seg * cps;
    double tot = 0.0;
    for (int c = 0; c < cps; ++c) tot += p[c];
    delta[(int64_t)blockIdx.y * delta_stride + seg] = sqrt(tot);
}

// p_l = Delta_l / sum Delta (Lemma 3.4), the level draw by the running sums of p, and the two thresholds of the drawn
// segment read off the sorted row.  One block per row.
__global__ void __launch_bounds__(1024)
stopk_sorted_draw_kernel(const uint32_t* __restrict__ sorted_rows, int64_t stride, const double* __restrict__ deltas,
                         int64_t delta_stride, int64_t d, int64_t s_len, int64_t L, int m0, uint64_t seed,
                         uint64_t step, double* p_all, double* u_dev, EmitParams* emit, Query* queries) {
    __shared__ double sh_sum[1024];
    __shared__ double sh_before[1025];
    __shared__ long long sh_last[1024];
    __shared__ long long sh_level, sh_jlast;
    __shared__ long long sh_pos[4];
    const int t = threadIdx.x;
    const int m = m0 + blockIdx.x;
    const uint32_t* sorted = sorted_rows + (int64_t)blockIdx.x * stride;
    const double* delta = deltas + (int64_t)blockIdx.x * delta_stride;
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
    __syncthreads();
    if (t == 0) {  // one running sum, so that the chunks tile [0, total] exactly
        double run = 0.0;
        long long j_last = -1;
        for (int i = 0; i < 1024; ++i) {
            sh_before[i] = run;
            run += sh_sum[i];
            j_last = max(j_last, sh_last[i]);
        }
        sh_before[1024] = run;
        sh_jlast = j_last;
        sh_level = -1;
    }
    __syncthreads();
    const double total = sh_before[1024], before = sh_before[t], end = sh_before[t + 1];
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
    int64_t level = (total > 0.0) ? (int64_t)sh_level : 0;
    if (level < 0) level = (sh_jlast >= 0) ? (int64_t)sh_jlast : 0;
    // the two ranks that bound the segment, and their thresholds from the sorted row (descending magnitude):
    // T = key of rank k, c = keys above it, n = keys equal to it.  Threads 0..3 search: (rank j, first / past).
    const int64_t kk[2] = {s_len * level, min(d, s_len * (level + 1))};
    if (t < 4) {
        const int64_t k = kk[t >> 1];
        long long pos = 0;
        if (k > 0 && k < d) {
            const uint32_t sk = sorted[k - 1];
            if ((t & 1) == 0) {  // first position holding sk
                int64_t lo = 0, hi = k - 1;
                while (lo < hi) {
                    const int64_t mid = (lo + hi) >> 1;
                    if (sorted[mid] < sk) lo = mid + 1; else hi = mid;
                }
                pos = lo;
            } else {  // first position past sk
                int64_t lo = k - 1, hi = d;
                while (lo < hi) {
                    const int64_t mid = (lo + hi) >> 1;
                    if (sorted[mid] <= sk) lo = mid + 1; else hi = mid;
                }
                pos = lo;
            }
        }
        sh_pos[t] = pos;
    }
    __syncthreads();
    if (t == 0) {
        u_dev[m] = u;
        p_all[m * kMaxLevels] = (total > 0.0) ? delta[level] / total : 1.0;
        emit[m].level = (int32_t)level;
    }
    if (t < 2) {
        const int64_t k = kk[t];
        Query q = {};
        q.k = (uint32_t)k;
        q.slot = kNoSlot;
        q.trivial = (k <= 0) ? 1u : (k >= d ? 2u : 0u);
        if (q.trivial == 1u) {
            q.T = kKeyNone;
        } else if (q.trivial == 2u) {
            q.T = 0u;
            q.r = 0xFFFFFFFFu;
        } else {
            const int64_t first = sh_pos[2 * t], past = sh_pos[2 * t + 1];
            q.T = kSortFlip - sorted[k - 1];
            q.c = (uint32_t)first;
            q.n = (uint32_t)(past - first);
            q.r = (uint32_t)(k - first);
        }
        queries[m * kMaxQueries + t] = q;
    }
}

struct SortLayout {
    int64_t nblocks;        // tiles per row
    int64_t table_words;    // per row
    int64_t partial_len;    // doubles per row
    size_t row_bytes;       // all buffers of one row
};

SortLayout sort_layout(int64_t d_max, int64_t big_cap) {
    SortLayout lay;
    lay.nblocks = (d_max + kSortTile - 1) / kSortTile;
    lay.table_words = 256 * lay.nblocks + 256;  // block counts per digit, and the digit totals
    lay.partial_len = 2 * (d_max / 1024) + 8;  // segments of >= 1024 keys: L * cps <= 1.5 d / 1024 + 1
    lay.row_bytes = sizeof(uint32_t) * (size_t)(2 * d_max + lay.table_words) + sizeof(double) * (size_t)(big_cap + lay.partial_len);
    return lay;
}

}  // namespace

int configure_sort_kernels() {  // the scatter's tile and tables pass 48 KB
    const int bytes = (int)(kScatterSmemWords * sizeof(uint32_t));
    if (cudaFuncSetAttribute(sort_scatter_kernel<SRC_KEYS>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
        cudaFuncSetAttribute(sort_scatter_kernel<SRC_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
        cudaFuncSetAttribute(sort_scatter_kernel<SRC_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return MLMC_OK;
}

// Rows that are sorted together, and the bytes of their buffers.
int stopk_sort_rows(int64_t d_max, int64_t big_cap, int M_max) {
    const SortLayout lay = sort_layout(d_max, big_cap);
    int64_t rows = (int64_t)(kSortScratchBudget / lay.row_bytes);
    if (rows < 1) rows = 1;
    if (rows > M_max) rows = M_max;
    return (int)rows;
}

size_t stopk_sort_scratch_bytes(int64_t d_max, int64_t big_cap, int M_max) {
    return sort_layout(d_max, big_cap).row_bytes * (size_t)stopk_sort_rows(d_max, big_cap, M_max);
}

// Sorts rows m0 .. m0 + rows - 1, computes their segment norms, draws their levels and fills their two queries.
void launch_stopk_sorted_rows(Workspace& ws, const void* g, int dtype, int64_t d, int m0, int rows, int64_t ld,
                              int64_t s_len, int64_t L, uint64_t seed, uint64_t step, cudaStream_t s) {
    const SortLayout lay = sort_layout(ws.d_max, ws.big_cap);
    const int cap = ws.sort_rows;
    uint32_t* buf_a = ws.sort_scratch;
    uint32_t* buf_b = buf_a + (int64_t)cap * ws.d_max;
    uint32_t* table = buf_b + (int64_t)cap * ws.d_max;
    uint32_t* totals = table + (int64_t)cap * 256 * lay.nblocks;
    double* delta = reinterpret_cast<double*>(table + (int64_t)cap * lay.table_words);  // 8-byte aligned: even word counts
    double* partial = delta + (int64_t)cap * ws.big_cap;
    const int nblocks = (int)((d + kSortTile - 1) / kSortTile);
    const dim3 grid((unsigned)nblocks, (unsigned)rows);
    const bool bf16 = dtype == MLMC_BF16;
    const int passes = bf16 ? 2 : 4;  // 15-bit and 31-bit keys
    const uint32_t* src = nullptr;
    uint32_t* dst = buf_a;
    for (int p = 0; p < passes; ++p) {
        const int shift = 8 * p;
        {
            LaunchScope t(ws, K_SORT_COUNT, s);
            if (p > 0)
                sort_count_kernel<SRC_KEYS><<<grid, kSortThreads, 0, s>>>(src, ws.d_max, d, shift, table, nblocks);
            else if (bf16)
                sort_count_kernel<SRC_BF16><<<grid, kSortThreads, 0, s>>>(
                    static_cast<const bf16_t*>(g) + (int64_t)m0 * ld, ld, d, shift, table, nblocks);
            else
                sort_count_kernel<SRC_F32><<<grid, kSortThreads, 0, s>>>(
                    static_cast<const float*>(g) + (int64_t)m0 * ld, ld, d, shift, table, nblocks);
        }
        {
            LaunchScope t(ws, K_SORT_SCAN, s);
            sort_scan_kernel<<<dim3(256, (unsigned)rows), 256, 0, s>>>(table, totals, nblocks);
        }
        {
            LaunchScope t(ws, K_SORT_SCATTER, s);
            if (p > 0)
                sort_scatter_kernel<SRC_KEYS><<<grid, kSortThreads, kScatterSmemWords * sizeof(uint32_t), s>>>(src, ws.d_max, dst, ws.d_max, d, shift,
                                                                             table, totals, nblocks);
            else if (bf16)
                sort_scatter_kernel<SRC_BF16><<<grid, kSortThreads, kScatterSmemWords * sizeof(uint32_t), s>>>(
                    static_cast<const bf16_t*>(g) + (int64_t)m0 * ld, ld, dst, ws.d_max, d, shift, table, totals, nblocks);
            else
                sort_scatter_kernel<SRC_F32><<<grid, kSortThreads, kScatterSmemWords * sizeof(uint32_t), s>>>(
                    static_cast<const float*>(g) + (int64_t)m0 * ld, ld, dst, ws.d_max, d, shift, table, totals, nblocks);
        }
        src = dst;
        dst = (dst == buf_a) ? buf_b : buf_a;
    }
    {
        LaunchScope t(ws, K_SEG_NORMS, s);
        if (s_len < 1024) {
            segment_norms_warp_kernel<<<dim3((unsigned)((L + 7) / 8), (unsigned)rows), 256, 0, s>>>(
                src, ws.d_max, d, s_len, L, bf16, delta, ws.big_cap);
        } else {
            const int cps = (int)((s_len + kNormChunk - 1) / kNormChunk);
            segment_chunk_energy_kernel<<<dim3((unsigned)(L * cps), (unsigned)rows), 256, 0, s>>>(
                src, ws.d_max, d, s_len, cps, bf16, partial, lay.partial_len);
            segment_finish_kernel<<<dim3((unsigned)((L + 255) / 256), (unsigned)rows), 256, 0, s>>>(
                partial, lay.partial_len, L, cps, delta, ws.big_cap);
        }
    }
    LaunchScope t(ws, K_STOPK_DRAW, s);
    stopk_sorted_draw_kernel<<<rows, 1024, 0, s>>>(src, ws.d_max, delta, ws.big_cap, d, s_len, L, m0, seed, step,
                                                   ws.p_all, ws.u_dev, ws.emit, ws.queries);
}

}  // namespace mlmc
