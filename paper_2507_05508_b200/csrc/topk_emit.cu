// Band emission (ordered stream compaction) and the server-side average for MLMC-Top-k.
//
// emit: writes the band of the drawn level of every worker,
//   { i : k_{l-1} < rank(i) <= k_l },  as (i, g_i / p_l) in ascending i  (Eq. 5 with g^0 = 0; Alg. 2 "Send").
// Membership is decided from the two thresholds (Ta, ra), (Tb, rb) of the band; equal-key elements
// are admitted by their index-ordered rank, so the position of an entry follows from the running counts
//   C = #{ Tb <= key <= Ta },  A = #{ key == Ta },  B = #{ key == Tb }
// over the elements before it.  The row is cut into tiles of kEmitTile 32-bit words, each of kEmitGroups batches;
// only the batches whose largest key (recorded by the first selection sweep) reaches Tb can hold band entries,
// the others are never read.  Four kernels, no waiting between thread blocks:
//   tile_list   one block per worker: the tiles that hold such a batch, each with the mask of those batches;
//   band_count  one warp per listed tile: the tile's C, A, B over its masked batches;
//   band_scan   one block per worker: exclusive running totals over the worker's listed tiles;
//   band_write  one warp per listed tile: reads the batches again and writes their entries at their final positions.
//
// aggregate: the dense mean (1/M) sum_m g~_m (Alg. 2 "Server aggregates") tiled over the index
// space; because every message is index-sorted, a tile's entries are one contiguous range per
// worker; they are added into a shared-memory tile in worker order and the tile is written once.
#include <atomic>

#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kBandThreads = 256;               // 8 warps per block, one tile per warp at a time
constexpr int kBatchWords = kEmitRows * 32;     // words a warp holds in registers at a time
static_assert(kEmitTile / kBatchWords == kEmitGroups, "a tile is kEmitGroups batches");
constexpr int kWriteSlots = 3;                  // shared-memory batches per warp of the write pass

// How a 32-bit word of the gradient row maps to elements: one fp32 element, or two bf16 elements
// (low half first).  A word past the end of the row reads as kPad, whose keys lie above every
// threshold the kernels use (thresholds are clamped to kCap, the key of +Inf), so padded elements
// are never inside the band.
template <typename T>
struct EmitWord;

template <>
struct EmitWord<float> {
    static constexpr int S = 1;
    static constexpr uint32_t kPad = 0x7FFFFFFFu;
    static constexpr uint32_t kCap = 0x7F800000u;
    __device__ static __forceinline__ uint32_t key(uint32_t w, int) { return w & 0x7FFFFFFFu; }
    __device__ static __forceinline__ float value(uint32_t w, int) { return __uint_as_float(w); }
};

template <>
struct EmitWord<bf16_t> {
    static constexpr int S = 2;
    static constexpr uint32_t kPad = 0x7FFF7FFFu;
    static constexpr uint32_t kCap = 0x7F80u;
    __device__ static __forceinline__ uint32_t key(uint32_t w, int s) { return s ? ((w >> 16) & 0x7FFFu) : (w & 0x7FFFu); }
    __device__ static __forceinline__ float value(uint32_t w, int s) {
        return __uint_as_float(s ? (w & 0xFFFF0000u) : (w << 16));
    }
};

// Number of band entries among a prefix of the row that holds C closed-range keys, A keys equal to Ta
// and B keys equal to Tb: the first min(A, ra) ties of Ta belong to Top-k_{l-1} (not to the band), and
// only the first min(B, rb) ties of Tb belong to Top-k_l.
__device__ __forceinline__ uint32_t band_prefix(uint32_t C, uint32_t A, uint32_t B, uint32_t ra, uint32_t rb) {
    return C - B + min(B, rb) - min(A, ra);
}

// Lane `lane` of a warp loads word i * 32 + lane (i < kEmitRows) of batch `batch` of tile `tile`: every row
// is one coalesced 128-byte request.  Words past the end of the row read as kPad.
template <typename T>
__device__ __forceinline__ void load_batch(const T* __restrict__ row, int64_t d, int64_t tile, int batch, int lane,
                                           uint32_t (&w)[kEmitRows]) {
    using EW = EmitWord<T>;
    const int64_t w0 = tile * kEmitTile + (int64_t)batch * kBatchWords + lane;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(row) + w0;
    if ((w0 - lane + kBatchWords) * EW::S <= d) {
#pragma unroll
        for (int i = 0; i < kEmitRows; ++i) w[i] = __ldg(words + i * 32);
    } else {
#pragma unroll
        for (int i = 0; i < kEmitRows; ++i) {
            const int64_t wi = w0 + i * 32;
            uint32_t v = EW::kPad;
            if ((wi + 1) * EW::S <= d) {
                v = __ldg(words + i * 32);
            } else if (EW::S == 2 && wi * 2 < d) {  // odd bf16 tail: only the low half exists
                v = (uint32_t)reinterpret_cast<const uint16_t*>(row)[wi * 2] | 0x7FFF0000u;
            }
            w[i] = v;
        }
    }
}

// The write pass gives every lane 16 consecutive words of a batch (four 16-byte chunks), so that the order of the
// lanes is the order of the coordinates.  Chunk c = 4 * lane + j of the batch is kept at position swz(c) of the
// warp's shared-memory slot: with the two low bits of the chunk number XOR-ed with bits 3..4, the eight lanes of a
// quarter warp read their j-th chunks (128-bit loads, 64 bytes apart before the swizzle) from eight different
// 16-byte bank groups.
__device__ __forceinline__ int swz(int c) { return (c & ~3) | ((c ^ (c >> 3)) & 3); }

// Starts the copy of batch `batch` of tile `tile` into a warp's shared-memory slot (kBatchWords words in the
// swizzled chunk order above): 16-byte asynchronous copies, or plain padded stores for the ragged end of the row.
template <typename T>
__device__ __forceinline__ void copy_batch_async(const T* __restrict__ row, int64_t d, int64_t tile, int batch, int lane,
                                                 uint32_t* slot) {
    using EW = EmitWord<T>;
    const int64_t w0 = tile * kEmitTile + (int64_t)batch * kBatchWords;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(row) + w0;
    if ((w0 + kBatchWords) * EW::S <= d) {
#pragma unroll
        for (int c = lane; c < kBatchWords / 4; c += 32) cp_async_16(slot + swz(c) * 4, words + c * 4);
    } else {
        for (int i = lane; i < kBatchWords; i += 32) {
            const int64_t wi = w0 + i;
            uint32_t v = EW::kPad;
            if ((wi + 1) * EW::S <= d) {
                v = __ldg(words + i);
            } else if (EW::S == 2 && wi * 2 < d) {  // odd bf16 tail: only the low half exists
                v = (uint32_t)reinterpret_cast<const uint16_t*>(row)[wi * 2] | 0x7FFF0000u;
            }
            slot[swz(i >> 2) * 4 + (i & 3)] = v;
        }
    }
}

// Closed-range flags of one batch and, per lane, its counts.  flags: bit i (fp32) or bits i and 16 + i
// (bf16 low / high half) = word i of this lane holds a key with Tb <= key <= Ta.  cA / cB: this lane's keys
// equal to Ta / Tb (looked for only when the warp has a closed-range key at all; ties are closed-range keys).
template <typename T>
__device__ __forceinline__ uint32_t batch_flags(const uint32_t (&w)[kEmitRows], uint32_t Tb, uint32_t Ta, uint32_t* cA,
                                                uint32_t* cB) {
    uint32_t flags = 0, a = 0, b = 0;
    if constexpr (EmitWord<T>::S == 1) {
        const uint32_t W = Ta - Tb;
#pragma unroll
        for (int i = 0; i < kEmitRows; ++i)
            if (((w[i] & 0x7FFFFFFFu) - Tb) <= W) flags |= 1u << i;
        if (__any_sync(0xFFFFFFFFu, flags != 0u)) {
#pragma unroll
            for (int i = 0; i < kEmitRows; ++i) {
                const uint32_t tk = (w[i] & 0x7FFFFFFFu) - Tb;
                a += (tk == W) ? 1u : 0u;
                b += (tk == 0u) ? 1u : 0u;
            }
        }
    } else {
        // two 15-bit keys per word; bit 15 of each half is free, so both halves are compared at
        // once: (key + 0x8000 - T) has bit 15 set iff key >= T, (T + 0x8000 - key) iff key <= T
        const uint32_t hi = 0x80008000u;
        const uint32_t geB = hi - Tb * 0x10001u, geB1 = hi - (Tb + 1u) * 0x10001u;
        const uint32_t leA = hi + Ta * 0x10001u, leA1 = hi + (Ta ? Ta - 1u : 0u) * 0x10001u;
        const uint32_t keepA1 = Ta ? 0xFFFFFFFFu : 0u;  // Ta = 0: every closed key equals Ta
        uint32_t acc = 0;
#pragma unroll
        for (int i = 0; i < kEmitRows; ++i) {
            const uint32_t k2 = w[i] & 0x7FFF7FFFu;
            flags |= ((k2 + geB) & (leA - k2) & hi) >> (15 - i);
        }
        if (__any_sync(0xFFFFFFFFu, flags != 0u)) {
#pragma unroll
            for (int i = 0; i < kEmitRows; ++i) {
                const uint32_t k2 = w[i] & 0x7FFF7FFFu;
                const uint32_t f = (k2 + geB) & (leA - k2) & hi;
                const uint32_t fB = f & ~(k2 + geB1);
                const uint32_t fA = f & ~((leA1 - k2) & keepA1);
                acc += (fA >> 15) + (fB >> 7);  // 5-bit counters: A at bits 0 / 16, B at bits 8 / 24
            }
        }
        a = (acc & 0x1Fu) + ((acc >> 16) & 0x1Fu);
        b = ((acc >> 8) & 0x1Fu) + ((acc >> 24) & 0x1Fu);
    }
    *cA = a;
    *cB = b;
    return flags;
}

// The same flags for the write pass, with the ties as masks instead of counts: bit i (fp32) or bits i and 16 + i
// (bf16 low / high half) of mA / mB = word i of this lane holds a key equal to Ta / Tb.
template <typename T>
__device__ __forceinline__ uint32_t batch_masks(const uint32_t (&w)[kEmitRows], uint32_t Tb, uint32_t Ta, bool ties,
                                                uint32_t* mA, uint32_t* mB) {
    uint32_t flags = 0, a = 0, b = 0;  // ties = false: the tile holds no key equal to a threshold, the masks stay empty
    if constexpr (EmitWord<T>::S == 1) {
        const uint32_t W = Ta - Tb;
#pragma unroll
        for (int i = 0; i < kEmitRows; ++i)
            if (((w[i] & 0x7FFFFFFFu) - Tb) <= W) flags |= 1u << i;
        if (ties && __any_sync(0xFFFFFFFFu, flags != 0u)) {
#pragma unroll
            for (int i = 0; i < kEmitRows; ++i) {
                const uint32_t tk = (w[i] & 0x7FFFFFFFu) - Tb;
                a |= (tk == W) ? (1u << i) : 0u;
                b |= (tk == 0u) ? (1u << i) : 0u;
            }
        }
    } else {
        const uint32_t hi = 0x80008000u;
        const uint32_t geB = hi - Tb * 0x10001u, geB1 = hi - (Tb + 1u) * 0x10001u;
        const uint32_t leA = hi + Ta * 0x10001u, leA1 = hi + (Ta ? Ta - 1u : 0u) * 0x10001u;
        const uint32_t keepA1 = Ta ? 0xFFFFFFFFu : 0u;  // Ta = 0: every closed key equals Ta
#pragma unroll
        for (int i = 0; i < kEmitRows; ++i) {
            const uint32_t k2 = w[i] & 0x7FFF7FFFu;
            flags |= ((k2 + geB) & (leA - k2) & hi) >> (15 - i);
        }
        if (ties && __any_sync(0xFFFFFFFFu, flags != 0u)) {
#pragma unroll
            for (int i = 0; i < kEmitRows; ++i) {
                const uint32_t k2 = w[i] & 0x7FFF7FFFu;
                const uint32_t f = (k2 + geB) & (leA - k2) & hi;
                b |= (f & ~(k2 + geB1)) >> (15 - i);
                a |= (f & ~((leA1 - k2) & keepA1)) >> (15 - i);
            }
        }
    }
    *mA = a;
    *mB = b;
    return flags;
}

// Flat numbering of the listed tiles of all workers (worker-major).  sh_off[m] = listed tiles of the workers
// before m; computed by the first warp of every block.
__device__ __forceinline__ void list_offsets(const uint32_t* __restrict__ tile_n, int M, uint32_t* sh_off) {
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        uint32_t carry = 0;
        for (int base = 0; base < M; base += 32) {
            const uint32_t n = (base + lane < M) ? tile_n[base + lane] : 0u;
            uint32_t incl = n;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += y;
            }
            if (base + lane < M) sh_off[base + lane] = carry + incl - n;
            carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        if (lane == 0) sh_off[M] = carry;
    }
    __syncthreads();
}

// Worker of flat entry f: the last m with sh_off[m] <= f (workers without listed tiles are skipped by the search).
__device__ __forceinline__ int worker_of(const uint32_t* sh_off, int M, uint32_t f) {
    int lo = 0, hi = M - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (sh_off[mid] <= f) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// The tiles of every worker that can hold band entries, ascending: a tile whose largest key is below the lower
// threshold Tb of the drawn band holds none (and no tie of Tb either), so the sweep leaves it out.
// One block per worker; every warp owns a contiguous range of tiles (a multiple of 32, so that its rows of 32 tiles
// are coalesced loads), counts its listed tiles, and after one barrier writes them behind those of the warps before.
constexpr int kListThreads = 1024;

__global__ void __launch_bounds__(kListThreads)
tile_list_kernel(const uint32_t* __restrict__ tile_max, int tiles_per_worker, const EmitParams* __restrict__ emit,
                 uint32_t key_cap, uint32_t* __restrict__ worker_tiles, uint32_t* __restrict__ tile_n,
                 uint32_t* __restrict__ group_n, int* status, int cached) {
    __shared__ uint32_t sh_warp[kListThreads / 32], sh_grp[kListThreads / 32];
    extern __shared__ uint8_t sh_mask[];  // [tiles_per_worker] batch masks of the counting pass, when they fit (cached != 0)
    const int m = blockIdx.x;
    const EmitParams e = emit[m];
    const bool on = e.enabled && e.level >= 0 && e.expect > 0u;
    const uint32_t Tb = min(e.Tb, key_cap);
    // the batch maxima of a tile are two 16-byte vectors; a batch below Tb holds no band entry and no tie of Tb
    const uint4* tmax = reinterpret_cast<const uint4*>(tile_max + (int64_t)m * tiles_per_worker * kEmitGroups);
    uint32_t* list = worker_tiles + (int64_t)m * tiles_per_worker;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rows = (tiles_per_worker + kListThreads - 1) / kListThreads;  // rows of 32 tiles per warp
    const int t0 = warp * rows * 32;
    auto batch_mask = [&](int t) -> uint32_t {
        if (t >= tiles_per_worker) return 0u;
        const uint4 a = __ldg(&tmax[2 * (int64_t)t]), b = __ldg(&tmax[2 * (int64_t)t + 1]);
        return (a.x >= Tb ? 1u : 0u) | (a.y >= Tb ? 2u : 0u) | (a.z >= Tb ? 4u : 0u) | (a.w >= Tb ? 8u : 0u) |
               (b.x >= Tb ? 16u : 0u) | (b.y >= Tb ? 32u : 0u) | (b.z >= Tb ? 64u : 0u) | (b.w >= Tb ? 128u : 0u);
    };
    uint32_t mine = 0, groups = 0;  // listed tiles of this warp (the same in every lane), batches of this lane
    if (on) {
#pragma unroll 4
        for (int r = 0; r < rows; ++r) {
            const int t = t0 + r * 32 + lane;
            const uint32_t bm = batch_mask(t);
            if (cached && t < tiles_per_worker) sh_mask[t] = (uint8_t)bm;  // read back by this same thread below
            mine += __popc(__ballot_sync(0xFFFFFFFFu, bm != 0u));
            groups += __popc(bm);
        }
    }
    groups = __reduce_add_sync(0xFFFFFFFFu, groups);
    if (lane == 0) {
        sh_warp[warp] = mine;
        sh_grp[warp] = groups;
    }
    __syncthreads();
    uint32_t before = 0, total = 0, total_groups = 0;
    for (int w = 0; w < kListThreads / 32; ++w) {
        const uint32_t x = sh_warp[w];
        total += x;
        total_groups += sh_grp[w];
        if (w < warp) before += x;
    }
    if (on && mine) {
        uint32_t pos = before;
        const uint32_t lt = (1u << lane) - 1u;
#pragma unroll 4
        for (int r = 0; r < rows; ++r) {
            const int t = t0 + r * 32 + lane;
            const uint32_t bm = cached ? (t < tiles_per_worker ? (uint32_t)sh_mask[t] : 0u) : batch_mask(t);
            const uint32_t mk = __ballot_sync(0xFFFFFFFFu, bm != 0u);
            if (bm) list[pos + __popc(mk & lt)] = (uint32_t)t | (bm << 24);  // tile numbers stay below 2^20
            pos += __popc(mk);
        }
    }
    if (threadIdx.x == 0) {
        tile_n[m] = total;
        group_n[m] = total_groups;
        if (on && total == 0u) set_status(status, MLMC_ERR_INTERNAL);  // a band with entries lies in some tile
    }
}

// Pass 1: C, A, B of every listed tile.  rec[m][j] = {C, A, B, 0} for the j-th listed tile of worker m.
template <typename T>
__global__ void __launch_bounds__(kBandThreads)
band_count_kernel(const T* __restrict__ g, int64_t d, int64_t ld, int tiles_per_worker,
                  const uint32_t* __restrict__ worker_tiles, const uint32_t* __restrict__ tile_n, int M,
                  const EmitParams* __restrict__ emit, uint4* __restrict__ rec) {
    using EW = EmitWord<T>;
    extern __shared__ uint32_t sh_off[];  // [M + 1]
    list_offsets(tile_n, M, sh_off);
    const uint32_t total = sh_off[M];
    const int lane = threadIdx.x & 31;
    const uint32_t warps = gridDim.x * (kBandThreads / 32);
    for (uint32_t f = blockIdx.x * (kBandThreads / 32) + (threadIdx.x >> 5); f < total; f += warps) {
        const int m = worker_of(sh_off, M, f);
        const uint32_t j = f - sh_off[m];
        const uint32_t entry = worker_tiles[(int64_t)m * tiles_per_worker + j];
        const int64_t tile = entry & 0xFFFFFFu;
        uint32_t todo = entry >> 24;  // the batches of the tile that can hold band entries (at least one)
        const uint32_t Tb = min(__ldg(&emit[m].Tb), EW::kCap), Ta = min(__ldg(&emit[m].Ta), EW::kCap);
        const T* row = g + (int64_t)m * ld;
        uint32_t cC = 0, cA = 0, cB = 0;
        uint32_t cur[kEmitRows], nxt[kEmitRows];
        load_batch<T>(row, d, tile, __ffs(todo) - 1, lane, cur);
        todo &= todo - 1u;
#pragma unroll 1
        for (bool more = true; more;) {
            more = todo != 0u;
            if (more) {  // in flight while this batch is counted
                load_batch<T>(row, d, tile, __ffs(todo) - 1, lane, nxt);
                todo &= todo - 1u;
            }
            uint32_t a1, b1;
            const uint32_t flags = batch_flags<T>(cur, Tb, Ta, &a1, &b1);
            cC += __popc(flags);
            cA += a1;
            cB += b1;
#pragma unroll
            for (int i = 0; i < kEmitRows; ++i) cur[i] = nxt[i];
        }
        const uint32_t totCA = __reduce_add_sync(0xFFFFFFFFu, cC | (cA << 16));  // at most 8192 elements per tile
        cB = __reduce_add_sync(0xFFFFFFFFu, cB);
        // the fourth word tells the write pass whether the tile holds a key equal to a threshold at all
        if (lane == 0)
            rec[(int64_t)m * tiles_per_worker + j] = make_uint4(totCA & 0xFFFFu, totCA >> 16, cB, ((totCA >> 16) | cB) ? 1u : 0u);
    }
}

// Pass 2: exclusive running totals over the listed tiles of every worker, in place, and the self-check that the
// band has exactly k_l - k_{l-1} entries.  One block per worker; every warp owns a contiguous range of the list (a
// multiple of 32 records, read as coalesced rows), adds it up, and after one barrier scans it row by row from the
// total of the warps before it.
__global__ void __launch_bounds__(kListThreads)
band_scan_kernel(uint4* __restrict__ rec, int tiles_per_worker, const uint32_t* __restrict__ tile_n,
                 const EmitParams* __restrict__ emit, int* status) {
    __shared__ uint32_t sh_w[3][kListThreads / 32];
    const int m = blockIdx.x;
    const int n = (int)tile_n[m];
    if (n == 0) return;
    uint4* r = rec + (int64_t)m * tiles_per_worker;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rows = (n + kListThreads - 1) / kListThreads;  // rows of 32 records per warp
    const int t0 = warp * rows * 32;
    uint32_t sC = 0, sA = 0, sB = 0;
#pragma unroll 4
    for (int i = 0; i < rows; ++i) {
        const int t = t0 + i * 32 + lane;
        if (t < n) {
            const uint4 x = r[t];
            sC += x.x; sA += x.y; sB += x.z;
        }
    }
    sC = __reduce_add_sync(0xFFFFFFFFu, sC);
    sA = __reduce_add_sync(0xFFFFFFFFu, sA);
    sB = __reduce_add_sync(0xFFFFFFFFu, sB);
    if (lane == 0) { sh_w[0][warp] = sC; sh_w[1][warp] = sA; sh_w[2][warp] = sB; }
    __syncthreads();
    uint32_t pC = 0, pA = 0, pB = 0, totC = 0, totA = 0, totB = 0;  // running totals before this warp's range
    for (int w = 0; w < kListThreads / 32; ++w) {
        const uint32_t xC = sh_w[0][w], xA = sh_w[1][w], xB = sh_w[2][w];
        totC += xC; totA += xA; totB += xB;
        if (w < warp) { pC += xC; pA += xA; pB += xB; }
    }
    for (int i = 0; i < rows; ++i) {
        const int t = t0 + i * 32 + lane;
        if (t0 + i * 32 >= n) break;  // warp-uniform
        uint4 x = make_uint4(0u, 0u, 0u, 0u);
        if (t < n) x = r[t];
        uint32_t iC = x.x, iA = x.y, iB = x.z;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t yC = __shfl_up_sync(0xFFFFFFFFu, iC, o), yA = __shfl_up_sync(0xFFFFFFFFu, iA, o),
                           yB = __shfl_up_sync(0xFFFFFFFFu, iB, o);
            if (lane >= o) { iC += yC; iA += yA; iB += yB; }
        }
        if (t < n) r[t] = make_uint4(pC + iC - x.x, pA + iA - x.y, pB + iB - x.z, x.w);
        pC += __shfl_sync(0xFFFFFFFFu, iC, 31);
        pA += __shfl_sync(0xFFFFFFFFu, iA, 31);
        pB += __shfl_sync(0xFFFFFFFFu, iB, 31);
    }
    if (threadIdx.x == 0) {
        const EmitParams e = emit[m];
        if (band_prefix(totC, totA, totB, e.ra, e.rb) != e.expect) set_status(status, MLMC_ERR_INTERNAL);
    }
}

// Pass 3: every listed tile is read again and its band entries are written at their final positions.
// A lane owns 16 consecutive words of a batch, so the order of the lanes is the order of the coordinates: the
// position of a lane's first entry is the batch's base plus the entries of the lanes before it (one warp scan per
// batch), and the lane then writes its own entries one after the other.
template <typename T>
__global__ void __launch_bounds__(kBandThreads, 4)
band_write_kernel(const T* __restrict__ g, int64_t d, int64_t ld, int tiles_per_worker,
                  const uint32_t* __restrict__ worker_tiles, const uint32_t* __restrict__ tile_n, int M,
                  const EmitParams* __restrict__ emit, const uint4* __restrict__ rec,
                  uint32_t* __restrict__ idx_out, float* __restrict__ val_out, int64_t capacity) {
    using EW = EmitWord<T>;
    constexpr int S = EW::S;
    static_assert(kEmitRows == 16, "a lane owns four 16-byte chunks of a batch");
    // every warp stages its batches in a ring of three shared-memory slots: two copies are in flight while a
    // batch is ranked, and the words of a batch can be addressed by a run-time index
    extern __shared__ __align__(16) uint32_t sh_dyn[];  // [warps][3][kBatchWords] ring, then sh_off[M + 1]
    uint32_t* sh_off = sh_dyn + (kBandThreads / 32) * kWriteSlots * kBatchWords;
    list_offsets(tile_n, M, sh_off);
    const uint32_t total = sh_off[M];
    const int lane = threadIdx.x & 31;
    uint32_t* ring = sh_dyn + (threadIdx.x >> 5) * kWriteSlots * kBatchWords;
    // where this lane's words sit in a slot: word r at own + (r ^ own_xor), i.e. chunk q at swz(4 * lane + q)
    const int own = lane * kEmitRows, own_xor = ((lane >> 1) & 3) << 2;
    const uint32_t warps = gridDim.x * (kBandThreads / 32);
    for (uint32_t f = blockIdx.x * (kBandThreads / 32) + (threadIdx.x >> 5); f < total; f += warps) {
        const int m = worker_of(sh_off, M, f);
        const uint32_t j = f - sh_off[m];
        const uint32_t entry = worker_tiles[(int64_t)m * tiles_per_worker + j];
        const int64_t tile = entry & 0xFFFFFFu;
        const EmitParams ep = emit[m];
        const uint32_t Tb = min(ep.Tb, EW::kCap), Ta = min(ep.Ta, EW::kCap);
        const uint32_t W = Ta - Tb;
        const float inv_p = (float)ep.inv_p;
        const T* row = g + (int64_t)m * ld;
        uint32_t* idx_w = idx_out + (int64_t)m * capacity;
        float* val_w = val_out + (int64_t)m * capacity;
        const uint4 pre = __ldg(&rec[(int64_t)m * tiles_per_worker + j]);
        uint32_t rC = pre.x, rA = pre.y, rB = pre.z;  // running totals before the current batch
        const bool tile_ties = pre.w != 0u;           // found by the count pass
        // Only the batches of the tile that can hold band entries are read (mask from the listing): `todo` walks them
        // for processing, `ahead` two batches further for the copies.
        uint32_t todo = entry >> 24, ahead = todo;
        __syncwarp();  // the previous tile's last batches have been read by every lane
        copy_batch_async<T>(row, d, tile, __ffs(ahead) - 1, lane, ring);
        ahead &= ahead - 1u;
        cp_async_commit();
        if (ahead) {
            copy_batch_async<T>(row, d, tile, __ffs(ahead) - 1, lane, ring + kBatchWords);
            ahead &= ahead - 1u;
        }
        cp_async_commit();
#pragma unroll 1
        for (int it = 0; todo; ++it) {
            const int b = __ffs(todo) - 1;
            todo &= todo - 1u;
            __syncwarp();  // the batch before this one has been read by every lane: its slot takes the copy two ahead
            if (ahead) {
                copy_batch_async<T>(row, d, tile, __ffs(ahead) - 1, lane, ring + ((it + 2) % kWriteSlots) * kBatchWords);
                ahead &= ahead - 1u;
            }
            cp_async_commit();  // one group per step, empty at the end of the tile
            cp_async_wait<2>();  // this batch has landed
            __syncwarp();
            const uint32_t* slot = ring + (it % kWriteSlots) * kBatchWords;
            uint32_t cur[kEmitRows];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 x = *reinterpret_cast<const uint4*>(slot + own + ((4 * q) ^ own_xor));
                cur[4 * q + 0] = x.x; cur[4 * q + 1] = x.y; cur[4 * q + 2] = x.z; cur[4 * q + 3] = x.w;
            }
            uint32_t mA, mB;
            uint32_t member = batch_masks<T>(cur, Tb, Ta, tile_ties, &mA, &mB);
            if (!__any_sync(0xFFFFFFFFu, member != 0u)) continue;  // no closed-range key in the batch: nothing to count either
            const uint32_t nC = __popc(member), nA = __popc(mA), nB = __popc(mB);
            const uint32_t totCA = __reduce_add_sync(0xFFFFFFFFu, nC | (nA << 16));
            const uint32_t myB = __reduce_add_sync(0xFFFFFFFFu, nB);
            const uint32_t myC = totCA & 0xFFFFu, myA = totCA >> 16;
            const uint32_t base = band_prefix(rC, rA, rB, ep.ra, ep.rb);
            if ((myA | myB) != 0u) {  // warp-uniform
                // Ties in this batch.  Unless the cut rank of a threshold falls among them, all of them are on one
                // side of it: the ties of Ta all outside Top-k_{l-1} (in the band) or all inside (dropped), the ties
                // of Tb all inside Top-k_l (in the band) or all outside (dropped).  Only a batch that holds a cut
                // ranks its ties one by one.
                const bool dropA = myA != 0u && rA + myA <= ep.ra, keepA = myA == 0u || rA >= ep.ra;
                const bool dropB = myB != 0u && rB >= ep.rb, keepB = myB == 0u || rB + myB <= ep.rb;
                const bool ranked = !((keepA || dropA) && (keepB || dropB)) || W == 0u;
                if (!ranked) {
                    if (dropA) member &= ~mA;
                    if (dropB) member &= ~mB;
                } else {
                    // index-ordered tie ranks (0-based): the ties of the lanes before this one, then this lane's in order
                    uint32_t iA = nA, iB = nB;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t yA = __shfl_up_sync(0xFFFFFFFFu, iA, o), yB = __shfl_up_sync(0xFFFFFFFFu, iB, o);
                        if (lane >= o) { iA += yA; iB += yB; }
                    }
                    uint32_t tA = rA + iA - nA, tB = rB + iB - nB;
                    const uint32_t t = mA | mB;
                    uint32_t rows = (S == 1) ? t : ((t | (t >> 16)) & 0xFFFFu);
                    while (rows) {
                        const int r = __ffs(rows) - 1;
                        rows &= rows - 1u;
#pragma unroll
                        for (int s = 0; s < S; ++s) {
                            const uint32_t bit = 1u << (r + 16 * s);
                            if (mA & bit) {
                                if (tA < ep.ra) member &= ~bit;   // still inside Top-k_{l-1}
                                ++tA;
                            }
                            if (mB & bit) {
                                if (tB >= ep.rb) member &= ~bit;  // already outside Top-k_l
                                ++tB;
                            }
                        }
                    }
                }
            }
            // positions: the batch's base plus the entries of the lanes before this one
            const uint32_t cnt = __popc(member);
            uint32_t incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += y;
            }
            uint32_t pos = base + incl - cnt;
            const uint32_t e0 = (uint32_t)((tile * kEmitTile + (int64_t)b * kBatchWords + lane * kEmitRows) * S);
            uint32_t rows = (S == 1) ? member : ((member | (member >> 16)) & 0xFFFFu);
            while (rows) {  // this lane's words that hold an entry, in ascending order
                const int r = __ffs(rows) - 1;
                rows &= rows - 1u;
                const uint32_t w = slot[own + (r ^ own_xor)];  // word r of this lane in the swizzled slot
#pragma unroll
                for (int s = 0; s < S; ++s) {
                    if ((member >> (r + 16 * s)) & 1u) {
                        if ((int64_t)pos < capacity) {
                            idx_w[pos] = e0 + (uint32_t)(r * S + s);
                            val_w[pos] = EW::value(w, s) * inv_p;
                        }
                        ++pos;
                    }
                }
            }
            rC += myC; rA += myA; rB += myB;
        }
    }
    cp_async_wait<0>();
}

// offsets[m][t] = first message entry of worker m whose index is >= t * kAggTile  (t = 0..ntiles)
__global__ void agg_offsets_kernel(const uint32_t* __restrict__ idx, const int64_t* __restrict__ count,
                                   const int32_t* __restrict__ level, int64_t capacity, int M, int ntiles,
                                   uint32_t* __restrict__ offsets) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)M * (ntiles + 1)) return;
    const int m = (int)(i / (ntiles + 1)), t = (int)(i % (ntiles + 1));
    const int64_t n = (level[m] < 0) ? 0 : count[m];
    const uint32_t* a = idx + (int64_t)m * capacity;
    const uint64_t target = (uint64_t)t * kAggTile;
    int64_t lo = 0, hi = n;
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((uint64_t)a[mid] < target) lo = mid + 1; else hi = mid;
    }
    offsets[i] = (uint32_t)lo;
}

// M is at most kEmitMaxWorkers: the offsets of all workers for one tile are fetched together.
__global__ void __launch_bounds__(256)
aggregate_topk_kernel(const uint32_t* __restrict__ idx, const float* __restrict__ val, int64_t capacity, int M,
                      int64_t d, int ntiles, const uint32_t* __restrict__ offsets, float* __restrict__ out) {
    __shared__ __align__(16) float acc[kAggTile];
    extern __shared__ uint32_t sh_off[];  // [2 M]: first and one-past-last message entry of every worker in this tile
    const float inv_M = 1.0f / (float)M;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t base = (int64_t)t * kAggTile;
        for (int i = threadIdx.x; i < 2 * M; i += blockDim.x)
            sh_off[i] = offsets[(int64_t)(i >> 1) * (ntiles + 1) + t + (i & 1)];
        for (int i = threadIdx.x; i < kAggTile / 4; i += blockDim.x)
            reinterpret_cast<float4*>(acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncthreads();
        for (int m = 0; m < M; ++m) {  // fixed worker order: reproducible fp32 sums
            const uint32_t o0 = sh_off[2 * m], o1 = sh_off[2 * m + 1];
            if (o1 > o0) {  // block-uniform
                const uint32_t* a = idx + (int64_t)m * capacity;
                const float* v = val + (int64_t)m * capacity;
                for (uint32_t j = o0 + threadIdx.x; j < o1; j += blockDim.x) {
                    const uint32_t off = a[j] - (uint32_t)base;  // indices are unique within a worker
                    if (off < (uint32_t)kAggTile) acc[off] += v[j];  // a message that is not index-sorted cannot reach outside the tile
                }
                __syncthreads();
            }
        }
        if (base + kAggTile <= d && (d & 3) == 0) {
            for (int i = threadIdx.x; i < kAggTile / 4; i += blockDim.x) {
                float4 x = reinterpret_cast<const float4*>(acc)[i];
                x.x *= inv_M; x.y *= inv_M; x.z *= inv_M; x.w *= inv_M;
                reinterpret_cast<float4*>(out + base)[i] = x;
            }
        } else {
            for (int i = threadIdx.x; i < kAggTile; i += blockDim.x)
                if (base + i < d) out[base + i] = acc[i] * inv_M;
        }
        __syncthreads();
    }
}


// The same average without a block barrier per worker: every warp owns kAggSub consecutive coordinates of the
// tile and adds the workers' entries that fall into them in worker order 0..M-1 (the order of the fp32 additions per
// coordinate is the same as in the kernel above, so the two give identical results).  Lane l finds, for worker
// m0 + l, where the warp's coordinates begin and end inside that worker's slice of the tile (two binary searches in
// an index-sorted slice); the warp then walks the workers one after the other.
constexpr int kAggSub = 512;
constexpr int kAggWarps = kAggTile / kAggSub;

__global__ void __launch_bounds__(kAggWarps * 32)
aggregate_topk_warps_kernel(const uint32_t* __restrict__ idx, const float* __restrict__ val, int64_t capacity, int M,
                            int64_t d, int ntiles, const uint32_t* __restrict__ offsets, float* __restrict__ out) {
    __shared__ __align__(16) float acc_all[kAggTile];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* acc = acc_all + warp * kAggSub;
    const float inv_M = 1.0f / (float)M;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t base = (int64_t)t * kAggTile + (int64_t)warp * kAggSub;  // first coordinate of this warp
#pragma unroll
        for (int i = 0; i < kAggSub / 128; ++i)
            reinterpret_cast<float4*>(acc)[i * 32 + lane] = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncwarp();
        if (base < d) {
            for (int m0 = 0; m0 < M; m0 += 32) {
                const int m = m0 + lane;
                uint32_t s0 = 0, s1 = 0;
                if (m < M) {
                    const uint32_t o0 = offsets[(int64_t)m * (ntiles + 1) + t], o1 = offsets[(int64_t)m * (ntiles + 1) + t + 1];
                    const uint32_t* a = idx + (int64_t)m * capacity;
                    auto first_at_least = [&](uint64_t target) -> uint32_t {
                        uint32_t lo = o0, hi = o1;
                        while (lo < hi) {
                            const uint32_t mid = lo + ((hi - lo) >> 1);
                            if ((uint64_t)__ldg(&a[mid]) < target) lo = mid + 1; else hi = mid;
                        }
                        return lo;
                    };
                    s0 = (warp == 0) ? o0 : first_at_least((uint64_t)base);
                    s1 = (warp == kAggWarps - 1) ? o1 : first_at_least((uint64_t)base + kAggSub);
                }
                const int nm = min(32, M - m0);
                for (int mm = 0; mm < nm; ++mm) {  // fixed worker order: reproducible fp32 sums
                    const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, s0, mm), b1 = __shfl_sync(0xFFFFFFFFu, s1, mm);
                    if (b1 > b0) {  // warp-uniform
                        const uint32_t* a = idx + (int64_t)(m0 + mm) * capacity;
                        const float* v = val + (int64_t)(m0 + mm) * capacity;
                        for (uint32_t j = b0 + lane; j < b1; j += 32) {
                            const uint32_t off = __ldg(&a[j]) - (uint32_t)base;  // indices are unique within a worker
                            if (off < (uint32_t)kAggSub) acc[off] += __ldg(&v[j]);  // an unsorted message cannot reach outside
                        }
                        __syncwarp();
                    }
                }
            }
        }
        if (base + kAggSub <= d && (d & 3) == 0) {
#pragma unroll
            for (int i = 0; i < kAggSub / 128; ++i) {
                float4 x = reinterpret_cast<const float4*>(acc)[i * 32 + lane];
                x.x *= inv_M; x.y *= inv_M; x.z *= inv_M; x.w *= inv_M;
                reinterpret_cast<float4*>(out + base)[i * 32 + lane] = x;
            }
        } else {
            for (int i = lane; i < kAggSub; i += 32)
                if (base + i < d) out[base + i] = acc[i] * inv_M;
        }
        __syncwarp();
    }
}

}  // namespace

int configure_emit_kernels() {  // the write pass: 48 KB ring + the list offsets of up to kEmitMaxWorkers workers
    const int smem = (kBandThreads / 32) * kWriteSlots * kBatchWords * (int)sizeof(uint32_t) +
                     (kEmitMaxWorkers + 1) * (int)sizeof(uint32_t);
    if (cudaFuncSetAttribute(tile_list_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(band_write_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
        cudaFuncSetAttribute(band_write_kernel<bf16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return MLMC_OK;
}

void launch_emit(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const mlmc_topk_msgs& out,
                 cudaStream_t s) {
    const int tpw = emit_tiles_per_worker(d, dtype);
    const int64_t most = (int64_t)tpw * M;  // listed tiles at most
    ws.last_emit_tiles = tpw;
    {
        LaunchScope t(ws, K_TILE_LIST, s);
        const int cached = tpw <= 96 * 1024;  // one byte per tile in shared memory
        tile_list_kernel<<<M, kListThreads, cached ? (size_t)tpw : 0, s>>>(
            ws.tile_max, tpw, ws.emit, dtype == MLMC_BF16 ? 0x7F80u : 0x7F800000u, ws.worker_tiles, ws.tile_n, ws.group_n,
            ws.status, cached);
    }
    const int wpb = kBandThreads / 32;
    const size_t smem = (size_t)(M + 1) * sizeof(uint32_t);
    const size_t smem_w = smem + (size_t)(kBandThreads / 32) * kWriteSlots * kBatchWords * sizeof(uint32_t);
    // grids of two whole waves: the warps take tiles with a grid stride, so a partial last wave costs a full one
    auto two_waves = [&](const void* kernel, size_t dyn_smem) -> int64_t {
        int resident = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kBandThreads, dyn_smem) != cudaSuccess || resident < 1)
            resident = 1;
        int64_t grid = (int64_t)ws.sm_count * resident * 2;
        const int64_t by_work = (most + wpb - 1) / wpb;
        return grid < by_work ? grid : by_work;
    };
    const bool bf = dtype == MLMC_BF16;
    const int64_t grid = two_waves(bf ? (const void*)band_count_kernel<bf16_t> : (const void*)band_count_kernel<float>, smem);
    const int64_t grid_w = two_waves(bf ? (const void*)band_write_kernel<bf16_t> : (const void*)band_write_kernel<float>, smem_w);
    {
        LaunchScope t(ws, K_BAND_COUNT, s);
        if (dtype == MLMC_BF16)
            band_count_kernel<bf16_t><<<(unsigned)grid, kBandThreads, smem, s>>>(
                static_cast<const bf16_t*>(g), d, ld, tpw, ws.worker_tiles, ws.tile_n, M, ws.emit, ws.tile_desc);
        else
            band_count_kernel<float><<<(unsigned)grid, kBandThreads, smem, s>>>(
                static_cast<const float*>(g), d, ld, tpw, ws.worker_tiles, ws.tile_n, M, ws.emit, ws.tile_desc);
    }
    {
        LaunchScope t(ws, K_BAND_SCAN, s);
        band_scan_kernel<<<M, kListThreads, 0, s>>>(ws.tile_desc, tpw, ws.tile_n, ws.emit, ws.status);
    }
    LaunchScope t(ws, K_EMIT, s);
    if (dtype == MLMC_BF16)
        band_write_kernel<bf16_t><<<(unsigned)grid_w, kBandThreads, smem_w, s>>>(
            static_cast<const bf16_t*>(g), d, ld, tpw, ws.worker_tiles, ws.tile_n, M, ws.emit, ws.tile_desc, out.idx,
            out.val, out.capacity);
    else
        band_write_kernel<float><<<(unsigned)grid_w, kBandThreads, smem_w, s>>>(
            static_cast<const float*>(g), d, ld, tpw, ws.worker_tiles, ws.tile_n, M, ws.emit, ws.tile_desc, out.idx,
            out.val, out.capacity);
}

void launch_aggregate_topk(Workspace& ws, const mlmc_topk_msgs& msgs, int M, int64_t d, float* out, cudaStream_t s) {
    const int ntiles = (int)((d + kAggTile - 1) / kAggTile);
    const int64_t n_off = (int64_t)M * (ntiles + 1);
    {
        LaunchScope t(ws, K_AGG_OFFSETS, s);
        agg_offsets_kernel<<<(unsigned)((n_off + 255) / 256), 256, 0, s>>>(msgs.idx, msgs.count, msgs.level,
                                                                           msgs.capacity, M, ntiles, ws.agg_offsets);
    }
    int grid = ws.sm_count * 8;
    if (grid > ntiles) grid = ntiles;
    LaunchScope t(ws, K_AGG_TOPK, s);
    aggregate_topk_warps_kernel<<<grid, kAggWarps * 32, 0, s>>>(msgs.idx, msgs.val, msgs.capacity, M, d, ntiles,
                                                                ws.agg_offsets, out);
}

}  // namespace mlmc

// ---------------------------------------------------------------------------------------------
// Server average of Top-k messages without any allocation.
// ---------------------------------------------------------------------------------------------
// The tile offsets that the averaging kernel needs normally live in the context's workspace, which
// mlmc_create obtains with cudaMalloc.  Here they live in a file-scope device array of fixed size,
// which every GPU that loads this library holds until the process exits.
namespace mlmc {
namespace {

constexpr int64_t kStaticOffsetWords = int64_t(1) << 20;  // 4 MiB: M * (ceil(d / kAggTile) + 1) entries at most
static __device__ __align__(256) uint32_t g_static_offsets[kStaticOffsetWords];

constexpr int kMaxDevices = 64;
// Device address of the array on each device, 0 = not looked up yet.  Host threads may make their first call on a
// device at the same time: the SM count is written first and the address is published last with a release store,
// so a thread that sees the address (acquire load) also sees the count.  Two threads that both find 0 look the
// same values up twice, which is harmless.
std::atomic<uint32_t*> g_static_offsets_addr[kMaxDevices];
int g_static_sm_count[kMaxDevices];

}  // namespace
}  // namespace mlmc

extern "C" int mlmc_aggregate_topk_noalloc(const mlmc_topk_msgs* msgs, int M, int64_t d, float* out, void* stream) {
    using namespace mlmc;
    if (!msgs || !out || !msgs->idx || !msgs->val || !msgs->count || !msgs->level) return MLMC_ERR_ARG;
    if (M < 1 || M > kEmitMaxWorkers || d < 1 || d >= (int64_t(1) << 32) || msgs->capacity < 0) return MLMC_ERR_ARG;
    const int64_t ntiles = (d + kAggTile - 1) / kAggTile;
    const int64_t n_off = (int64_t)M * (ntiles + 1);
    if (n_off > kStaticOffsetWords) return MLMC_ERR_ARG;  // beyond the fixed scratch: use mlmc_aggregate with a context
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MLMC_ERR_CUDA;
    uint32_t* offsets = g_static_offsets_addr[dev].load(std::memory_order_acquire);
    if (!offsets) {
        // Set-up, once per device, with that device current.  In host code the array's name only stands
        // for the symbol; the address a kernel can use has to be asked for.
        uint32_t* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_offsets) != cudaSuccess || !p) {
            cudaGetLastError();
            return MLMC_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            return MLMC_ERR_CUDA;
        g_static_sm_count[dev] = sms;
        g_static_offsets_addr[dev].store(p, std::memory_order_release);
        offsets = p;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // every entry in [0, n_off) is rewritten by this kernel, so nothing is left over from an earlier call
    agg_offsets_kernel<<<(unsigned)((n_off + 255) / 256), 256, 0, s>>>(msgs->idx, msgs->count, msgs->level,
                                                                       msgs->capacity, M, (int)ntiles, offsets);
    int64_t grid = (int64_t)g_static_sm_count[dev] * 8;
    if (grid > ntiles) grid = ntiles;
    aggregate_topk_kernel<<<(unsigned)grid, 256, 2 * M * sizeof(uint32_t), s>>>(msgs->idx, msgs->val, msgs->capacity, M, d,
                                                                                (int)ntiles, offsets, out);
    return cudaGetLastError() == cudaSuccess ? MLMC_OK : MLMC_ERR_CUDA;
}
