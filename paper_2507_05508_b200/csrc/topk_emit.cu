// Band emission (ordered stream compaction) and the server-side average for MLMC-Top-k.
//
// emit: one sweep over every worker's gradient writes the band of the drawn level,
//   { i : k_{l-1} < rank(i) <= k_l },  as (i, g_i / p_l) in ascending i  (Eq. 5 with g^0 = 0; Alg. 2 "Send").
// Membership is decided from the two thresholds (Ta, ra), (Tb, rb) of the band; equal-key elements
// are admitted by their index-ordered rank, so the running counts
//   C = #{ Tb <= key <= Ta },  A = #{ key == Ta },  B = #{ key == Tb }
// are carried across tiles with a decoupled look-back (tiles are numbered by a ticket counter, so
// every predecessor of a running tile has already started; every wait is bounded).
//
// aggregate: the dense mean (1/M) sum_m g~_m (Alg. 2 "Server aggregates") tiled over the index
// space; because every message is index-sorted, a tile's entries are one contiguous range per
// worker; they are added into a shared-memory tile in worker order and the tile is written once.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr unsigned kSpinLimit = 1u << 22;          // polls of a shared-memory word before a wait gives up
constexpr unsigned kLookbackSpinLimit = 1u << 20;  // polls of a look-back record (each poll is a global load)
constexpr int kTicketRing = 16;

// Look-back record of one tile: {C, A, B, state}: closed-range keys (Tb <= key <= Ta), keys equal to Ta,
// keys equal to Tb; state 0 = not yet, 1 = the tile's own counts, 2 = running totals up to and including
// the tile.  A record is written and read as one 16-byte access, so counts and state belong together.
__device__ __forceinline__ void put_record(uint4* rec, uint32_t C, uint32_t A, uint32_t B, uint32_t state) {
    __stcg(rec, make_uint4(C, A, B, state));
}

// How a 32-bit word of the gradient row maps to elements: one fp32 element, or two bf16 elements
// (low half first).  A word past the end of the row reads as kPad, whose keys lie above every
// threshold the kernel uses (thresholds are clamped to kCap, the key of +Inf), so padded elements
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

// Starts the copy of one warp's share (kEmitRows * 32 consecutive words) of tile t of a row into its
// share of a shared-memory slot.  Full tiles go as 16-byte asynchronous copies; the ragged last tile of
// a row is written with plain stores, padded with kPad.
template <typename T>
__device__ __forceinline__ void emit_fetch_share(const T* __restrict__ row, int64_t d, int64_t tile, uint32_t* share,
                                                 int warp, int lane) {
    using EW = EmitWord<T>;
    constexpr int kShare = kEmitRows * 32;
    const int64_t w0 = tile * kEmitTile + warp * kShare;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(row) + w0;
    if ((tile + 1) * kEmitTile * EW::S <= d) {
#pragma unroll
        for (int c = lane; c < kShare / 4; c += 32) cp_async_16(share + c * 4, words + c * 4);
    } else {
        for (int i = lane; i < kShare; i += 32) {
            const int64_t wi = w0 + i;
            uint32_t v = EW::kPad;
            if ((wi + 1) * EW::S <= d) {
                v = __ldg(words + i);
            } else if (EW::S == 2 && wi * 2 < d) {  // odd bf16 tail: only the low half exists
                v = (uint32_t)reinterpret_cast<const uint16_t*>(row)[wi * 2] | 0x7FFF0000u;
            }
            share[i] = v;
        }
    }
}

// Block-local hand-over words between the worker warps and the prefix warp.  All counters only grow.
struct EmitSync {
    unsigned tickets_ready;         // tickets [0, tickets_ready) of this block are in the ticket ring
    unsigned counted[kEmitStages];  // per slot: worker warps that have posted counts (kEmitWorkers more per tile;
                                    // per slot, because a fast warp may count tile k+1 before a slow one counts tile k)
    unsigned ready[kEmitStages];    // per slot: j + 1 once tile j of this block has its prefix in shared memory
    int abort;                      // a bounded wait gave up: everybody leaves
};

__device__ __forceinline__ unsigned ld_volatile_shared(const unsigned* p) { return *reinterpret_cast<const volatile unsigned*>(p); }

// The whole warp spins until *p >= want (bounded).  Returns false, for every lane alike, when the wait
// gave up (which raises the block's abort flag) or another warp had raised it.
__device__ __forceinline__ bool wait_at_least(const unsigned* p, unsigned want, int* abort_flag) {
    unsigned spins = 0;
    bool ok = true;
    while (ld_volatile_shared(p) < want) {
        if (*reinterpret_cast<volatile int*>(abort_flag)) {
            ok = false;
            break;
        }
        if (++spins > kSpinLimit) {
            *reinterpret_cast<volatile int*>(abort_flag) = 1;
            ok = false;
            break;
        }
        __nanosleep(64);  // a waiting warp leaves the issue slots to the warps that have work
    }
    ok = __all_sync(0xFFFFFFFFu, ok);
    return ok;
}

// Persistent blocks take tiles in ticket order; consecutive tickets go to different workers (ticket q is
// tile q / M of worker q % M).  Eight worker warps each own a fixed share of every tile; a ninth warp
// owns the tickets and the prefixes, so nobody waits at a block-wide barrier:
//   worker, iteration k:  count its share of tile k (closed-range keys Tb <= key <= Ta, ties of Ta and Tb),
//                         write its share of tile k-2 at the final positions (within a warp row the band
//                         entries are consecutive, so the stores coalesce), start the copy of tile k+2;
//   prefix warp, tile j:  when all shares of tile j are counted, publish the tile's counts; then finish
//                         tile j-1: sum the records of the worker's earlier tiles (decoupled look-back)
//                         and hand the prefix to the workers.
// Every wait is bounded; a wait that gives up sets MLMC_ERR_TIMEOUT and makes the block leave.
template <typename T>
__global__ void __launch_bounds__(kEmitThreads, kEmitBlocksPerSM)
emit_kernel(const T* __restrict__ g, int64_t d, int64_t ld, int tiles_per_worker, unsigned total_tiles, int M,
            const EmitParams* __restrict__ emit, uint4* tile_desc, unsigned* tile_counter,
            uint32_t* __restrict__ idx_out, float* __restrict__ val_out, int64_t capacity, int* status,
            int* worker_err) {
    using EW = EmitWord<T>;
    constexpr int S = EW::S;
    constexpr int kShare = kEmitRows * 32;
    extern __shared__ __align__(16) uint32_t sh_ring[];  // [kEmitStages][kEmitTile]
    __shared__ EmitSync sy;
    // The hand-over data is volatile and is published by a volatile flag store (or a shared-memory atomic) issued
    // after it by the same thread: shared-memory accesses of one warp are performed in program order, so no fence
    // is used (a fence would also wait for the asynchronous tile copies and the ticket atomic still in flight).
    __shared__ volatile unsigned sh_ticket[kTicketRing];          // tile k of this block: its ticket q ...
    __shared__ volatile int sh_tm[kTicketRing], sh_tt[kTicketRing];  // ... its worker q % M and its tile index q / M
    // The counts of a tile are read by the workers when they write it, two iterations after counting; a fast warp
    // may by then count the tile four ahead of a slow warp's write, so the counts keep eight tiles, not four.
    constexpr int kCountSlots = 2 * kEmitStages;
    __shared__ volatile uint32_t sh_cC[kCountSlots][kEmitWorkers], sh_cA[kCountSlots][kEmitWorkers], sh_cB[kCountSlots][kEmitWorkers];
    __shared__ volatile uint32_t sh_pre[kEmitStages][4];  // {C, A, B} before the tile; [3]: 1 = valid, 0 = skip the write
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const unsigned kNone = 0xFFFFFFFFu;
    // the band parameters of every worker, copied once (the ring is followed by M of them)
    EmitParams* sh_emit = reinterpret_cast<EmitParams*>(sh_ring + kEmitStages * kEmitTile);
    for (int i = threadIdx.x; i < M * (int)(sizeof(EmitParams) / 4); i += kEmitThreads)
        reinterpret_cast<uint32_t*>(sh_emit)[i] = reinterpret_cast<const uint32_t*>(emit)[i];

    if (threadIdx.x == 0) {
        sy.tickets_ready = 0; sy.abort = 0;
        for (int i = 0; i < kEmitStages; ++i) sy.counted[i] = sy.ready[i] = 0;
    }
    __syncthreads();

    if (warp < kEmitWorkers) {
        // =========================== worker warps ===========================
        uint32_t* my_ring = sh_ring + warp * kShare;
        auto fetch = [&](unsigned q, int k) {  // one commit per call, also for tiles that are skipped
            if (q < total_tiles) {
                const int mq = sh_tm[k & (kTicketRing - 1)];
                if (sh_emit[mq].enabled)
                    emit_fetch_share<T>(g + (int64_t)mq * ld, d, (int64_t)sh_tt[k & (kTicketRing - 1)],
                                        my_ring + (k & (kEmitStages - 1)) * kEmitTile, warp, lane);
            }
            cp_async_commit();
        };
        auto ticket_of = [&](int k, unsigned* q) -> bool {
            if (!wait_at_least(&sy.tickets_ready, (unsigned)k + 1u, &sy.abort)) return false;
            *q = sh_ticket[k & (kTicketRing - 1)];
            return true;
        };
        unsigned q_m2 = kNone, q_m1 = kNone, q_0 = kNone, q_p1 = kNone;  // tiles k-2, k-1, k, k+1
        uint32_t fl_m2 = 0, fl_m1 = 0, ra_m2 = 0, ra_m1 = 0;              // their flags / row masks
        // Worker warp 0 owns the tickets: one per iteration, for the tile three ahead, so every ticket is taken
        // the same short time before its tile is counted and the tiles start in ticket order across the grid.
        bool more = true;  // valid tickets may remain
        auto put_ticket = [&](unsigned i, unsigned q) {
            if (q >= total_tiles) {
                q = kNone;
                more = false;
            }
            if (lane == 0) {
                sh_tm[i & (kTicketRing - 1)] = (int)(q % (unsigned)M);  // divided once here, read by every warp
                sh_tt[i & (kTicketRing - 1)] = (int)(q / (unsigned)M);
                sh_ticket[i & (kTicketRing - 1)] = q;
                *reinterpret_cast<volatile unsigned*>(&sy.tickets_ready) = i + 1u;
            }
        };
        if (warp == 0) {
            unsigned base = 0;
            if (lane == 0) base = atomicAdd(tile_counter, 3u);
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            for (unsigned i = 0; i < 3u; ++i) put_ticket(i, base + i);
        }
        bool alive = ticket_of(0, &q_0) && ticket_of(1, &q_p1);
        if (alive) {
            fetch(q_0, 0);
            fetch(q_p1, 1);
        }
        for (int k = 0; alive && (q_0 < total_tiles || q_m2 < total_tiles || q_m1 < total_tiles); ++k) {
            // the ticket of tile k+3 is asked for now and handed out at the end of the iteration
            unsigned q_new = kNone;
            if (warp == 0 && more && lane == 0) q_new = atomicAdd(tile_counter, 1u);

            // ---- count this warp's share of tile k.
            // flags: bit i (fp32) or bits i and 16 + i (bf16 low / high half) = word i holds a closed-range key
            uint32_t flags = 0, rowany = 0;
            if (q_0 < total_tiles) {
                const int mc_ = sh_tm[k & (kTicketRing - 1)];
                const EmitParams ec = sh_emit[mc_];
                uint32_t cC = 0, cA = 0, cB = 0;
                cp_async_wait<1>();  // the share of tile k has landed (tile k+1 may still be in flight)
                __syncwarp();
                if (ec.enabled) {
                    const uint32_t* tile = my_ring + (k & (kEmitStages - 1)) * kEmitTile + lane;
                    const uint32_t Tb = min(ec.Tb, EW::kCap), Ta = min(ec.Ta, EW::kCap);
                    if constexpr (S == 1) {
                        const uint32_t W = Ta - Tb;
#pragma unroll
                        for (int i = 0; i < kEmitRows; ++i)
                            if (((tile[i * 32] & 0x7FFFFFFFu) - Tb) <= W) flags |= 1u << i;
                        if (__any_sync(0xFFFFFFFFu, flags != 0u)) {  // ties are closed-range keys: look only if there are any
#pragma unroll
                            for (int i = 0; i < kEmitRows; ++i) {
                                const uint32_t tk = (tile[i * 32] & 0x7FFFFFFFu) - Tb;
                                cA += (tk == W) ? 1u : 0u;
                                cB += (tk == 0u) ? 1u : 0u;
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
                            const uint32_t k2 = tile[i * 32] & 0x7FFF7FFFu;
                            flags |= ((k2 + geB) & (leA - k2) & hi) >> (15 - i);
                        }
                        if (__any_sync(0xFFFFFFFFu, flags != 0u)) {  // ties are closed-range keys: look only if there are any
#pragma unroll
                            for (int i = 0; i < kEmitRows; ++i) {
                                const uint32_t k2 = tile[i * 32] & 0x7FFF7FFFu;
                                const uint32_t f = (k2 + geB) & (leA - k2) & hi;
                                const uint32_t fB = f & ~(k2 + geB1);
                                const uint32_t fA = f & ~((leA1 - k2) & keepA1);
                                acc += (fA >> 15) + (fB >> 7);  // 5-bit counters: A at bits 0 / 16, B at bits 8 / 24
                            }
                        }
                        cA = (acc & 0x1Fu) + ((acc >> 16) & 0x1Fu);
                        cB = ((acc >> 8) & 0x1Fu) + ((acc >> 24) & 0x1Fu);
                    }
                    rowany = __reduce_or_sync(0xFFFFFFFFu, flags);
                    if (rowany) {
                        const uint32_t totCA = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)__popc(flags) | (cA << 16));
                        cB = __reduce_add_sync(0xFFFFFFFFu, cB);
                        cC = totCA & 0xFFFFu;
                        cA = totCA >> 16;
                    }
                }
                // post the counts; the warp that posts last publishes the tile's record at once
                const int cs = k & (kCountSlots - 1);
                unsigned last = 0;
                if (lane == 0) {
                    sh_cC[cs][warp] = cC; sh_cA[cs][warp] = cA; sh_cB[cs][warp] = cB;
                    last = (atomicAdd(&sy.counted[k & (kEmitStages - 1)], 1u) + 1u ==
                            ((unsigned)k / kEmitStages + 1u) * kEmitWorkers) ? 1u : 0u;
                }
                if (__shfl_sync(0xFFFFFFFFu, last, 0) && ec.enabled) {
                    const uint32_t aggC = __reduce_add_sync(0xFFFFFFFFu, (lane < kEmitWorkers) ? sh_cC[cs][lane] : 0u);
                    const uint32_t aggA = __reduce_add_sync(0xFFFFFFFFu, (lane < kEmitWorkers) ? sh_cA[cs][lane] : 0u);
                    const uint32_t aggB = __reduce_add_sync(0xFFFFFFFFu, (lane < kEmitWorkers) ? sh_cB[cs][lane] : 0u);
                    const int tc = sh_tt[k & (kTicketRing - 1)];
                    // a worker's first tile has nothing before it: its counts are already running totals
                    if (lane == 0)
                        put_record(&tile_desc[(int64_t)mc_ * tiles_per_worker + tc], aggC, aggA, aggB, tc == 0 ? 2u : 1u);
                }
            }

            // ---- write this warp's share of tile k-2
            if (q_m2 < total_tiles) {
                const int mp = sh_tm[(k - 2) & (kTicketRing - 1)], tp = sh_tt[(k - 2) & (kTicketRing - 1)];
                const EmitParams ep = sh_emit[mp];
                const int slot = (k - 2) & (kEmitStages - 1);
                if (!wait_at_least(&sy.ready[slot], (unsigned)(k - 2) + 1u, &sy.abort)) {
                    alive = false;
                    break;
                }
                if (ep.enabled && ra_m2 && sh_pre[slot][3]) {
                    const uint32_t* tile = my_ring + slot * kEmitTile + lane;
                    const uint32_t Tb = min(ep.Tb, EW::kCap);
                    const uint32_t W = min(ep.Ta, EW::kCap) - Tb;
                    // counts of the warps before this one in the tile (every warp of the tile has posted: the prefix is out)
                    const int cs = (k - 2) & (kCountSlots - 1);
                    const uint32_t wC = __reduce_add_sync(0xFFFFFFFFu, (lane < warp) ? sh_cC[cs][lane] : 0u);
                    const uint32_t wA = __reduce_add_sync(0xFFFFFFFFu, (lane < warp) ? sh_cA[cs][lane] : 0u);
                    const uint32_t wB = __reduce_add_sync(0xFFFFFFFFu, (lane < warp) ? sh_cB[cs][lane] : 0u);
                    uint32_t rA = sh_pre[slot][1] + wA, rB = sh_pre[slot][2] + wB;
                    uint32_t base = band_prefix(sh_pre[slot][0] + wC, rA, rB, ep.ra, ep.rb);
                    // ties in this warp's share?  (warp-uniform; ties elsewhere only move the base)
                    // Ties in this warp's share (warp-uniform; ties elsewhere only move the base).  Unless the cut
                    // rank of a threshold falls among this share's ties, all of them are on one side of it: the
                    // ties of Ta all outside Top-k_{l-1} (in the band) or all inside (dropped), the ties of Tb all
                    // inside Top-k_l (in the band) or all outside (dropped).  Only the share that holds a cut
                    // ranks its ties one by one.
                    const uint32_t myA = sh_cA[cs][warp], myB = sh_cB[cs][warp];
                    const bool dropA = myA != 0u && rA + myA <= ep.ra, keepA = myA == 0u || rA >= ep.ra;
                    const bool dropB = myB != 0u && rB >= ep.rb, keepB = myB == 0u || rB + myB <= ep.rb;
                    const bool ties = !((keepA || dropA) && (keepB || dropB)) || ((myA | myB) != 0u && W == 0u);
                    const bool drop_any = !ties && (dropA || dropB);
                    const float inv_p = (float)ep.inv_p;
                    uint32_t* idx_w = idx_out + (int64_t)mp * capacity;
                    float* val_w = val_out + (int64_t)mp * capacity;
                    const uint32_t e0 = (uint32_t)(((int64_t)tp * kEmitTile + warp * kShare + lane) * S);
                    uint32_t rows = (ra_m2 | (ra_m2 >> 16)) & 0xFFFFu;  // rows that hold a closed-range key
                    // rolled loops over the rows that matter: the body is long, unrolling it 16 times would not fit
                    // the instruction cache
#pragma unroll 1
                    while (rows) {
                        const int i = __ffs(rows) - 1;
                        rows &= rows - 1u;
                        const uint32_t w = tile[i * 32];
                        bool em[S];
                        uint32_t me[S];
                        if (!ties) {
#pragma unroll
                            for (int s = 0; s < S; ++s) {
                                em[s] = (fl_m2 >> (i + 16 * s)) & 1u;
                                if (drop_any) {  // warp-uniform
                                    const uint32_t tk = EW::key(w, s) - Tb;
                                    em[s] = em[s] && !(dropA && tk == W) && !(dropB && tk == 0u);
                                }
                                me[s] = __ballot_sync(0xFFFFFFFFu, em[s]);
                            }
                        } else {
                            uint32_t tk[S], mA[S], mB[S], a_lt = 0, b_lt = 0;
#pragma unroll
                            for (int s = 0; s < S; ++s) {
                                tk[s] = EW::key(w, s) - Tb;
                                mA[s] = __ballot_sync(0xFFFFFFFFu, tk[s] == W);
                                mB[s] = __ballot_sync(0xFFFFFFFFu, tk[s] == 0u);
                                a_lt += __popc(mA[s] & lt);
                                b_lt += __popc(mB[s] & lt);
                            }
#pragma unroll
                            for (int s = 0; s < S; ++s) {
                                // index-ordered tie ranks (0-based) of this element among the keys equal to Ta / Tb
                                const bool inA = (tk[s] == W) && (rA + a_lt) < ep.ra;    // still inside Top-k_{l-1}
                                const bool outB = (tk[s] == 0u) && (rB + b_lt) >= ep.rb; // already outside Top-k_l
                                em[s] = (tk[s] <= W) && !inA && !outB;
                                me[s] = __ballot_sync(0xFFFFFFFFu, em[s]);
                                a_lt += (mA[s] >> lane) & 1u;
                                b_lt += (mB[s] >> lane) & 1u;
                            }
#pragma unroll
                            for (int s = 0; s < S; ++s) {
                                rA += __popc(mA[s]);
                                rB += __popc(mB[s]);
                            }
                        }
                        uint32_t pos = base;
#pragma unroll
                        for (int s = 0; s < S; ++s) pos += __popc(me[s] & lt);
#pragma unroll
                        for (int s = 0; s < S; ++s) {
                            if (em[s]) {
                                if ((int64_t)pos < capacity) {
                                    idx_w[pos] = e0 + (uint32_t)(i * 32 * S + s);
                                    val_w[pos] = EW::value(w, s) * inv_p;
                                }
                                ++pos;
                            }
                        }
                        base = __shfl_sync(0xFFFFFFFFu, pos, 31);  // lane 31 ends at the row's total
                    }
                }
            }

            if (warp == 0) put_ticket((unsigned)k + 3u, __shfl_sync(0xFFFFFFFFu, q_new, 0));

            // ---- start the copy of tile k+2 into the slot that tile k-2 has just left
            unsigned q_p2 = kNone;
            if (!ticket_of(k + 2, &q_p2)) {
                alive = false;
                break;
            }
            __syncwarp();
            fetch(q_p2, k + 2);
            q_m2 = q_m1; q_m1 = q_0; q_0 = q_p1; q_p1 = q_p2;
            fl_m2 = fl_m1; fl_m1 = flags;
            ra_m2 = ra_m1; ra_m1 = rowany;
        }
        cp_async_wait<0>();
    } else {
        // =========================== prefix warps ===========================
        // Two warps share the tiles of the block: warp pw handles tiles pw, pw + 2, ...  A tile's counts are
        // published by the worker warp that posts last (nothing delays them); a prefix warp looks back for
        // tile j once the block's next tile j+1 is counted too: by then the tiles that were counted at about
        // the same time as tile j have published their counts, and the tiles one round of the grid earlier
        // have their running totals, so the nearest running total lies inside the 128-record window.
        const int pw = warp - kEmitWorkers;
        constexpr int kWin = 4;  // look-back records per lane and step
        for (unsigned j = (unsigned)pw;; j += 2) {
            if (!wait_at_least(&sy.tickets_ready, j + 2u, &sy.abort)) break;  // tickets j and j+1 are out
            const unsigned q = sh_ticket[j & (kTicketRing - 1)], q_next = sh_ticket[(j + 1u) & (kTicketRing - 1)];
            if (q >= total_tiles) break;  // tickets only grow: nothing valid follows
            const int m = sh_tm[j & (kTicketRing - 1)], t = sh_tt[j & (kTicketRing - 1)];
            const int slot = (int)(j & (kEmitStages - 1));
            if (!wait_at_least(&sy.counted[slot], (j / kEmitStages + 1u) * kEmitWorkers, &sy.abort)) break;
            if (q_next < total_tiles &&
                !wait_at_least(&sy.counted[(j + 1u) & (kEmitStages - 1)], ((j + 1u) / kEmitStages + 1u) * kEmitWorkers, &sy.abort))
                break;
            const EmitParams& e = sh_emit[m];
            uint32_t pC = 0, pA = 0, pB = 0;
            bool ok = true;
            if (e.enabled) {
                uint4* desc = tile_desc + (int64_t)m * tiles_per_worker;
                const int cs = (int)(j & (kCountSlots - 1));
                const uint32_t aggC = __reduce_add_sync(0xFFFFFFFFu, (lane < kEmitWorkers) ? sh_cC[cs][lane] : 0u);
                const uint32_t aggA = __reduce_add_sync(0xFFFFFFFFu, (lane < kEmitWorkers) ? sh_cA[cs][lane] : 0u);
                const uint32_t aggB = __reduce_add_sync(0xFFFFFFFFu, (lane < kEmitWorkers) ? sh_cB[cs][lane] : 0u);
                if (t > 0) {
                    // lane i holds tiles look - i - 32 w; positions before the worker's first tile are an empty running total
                    uint4 rec[kWin];
                    int look = t - 1;
#pragma unroll
                    for (int w = 0; w < kWin; ++w) {
                        const int at = look - lane - 32 * w;
                        rec[w] = (at >= 0) ? __ldcg(&desc[at]) : make_uint4(0u, 0u, 0u, 2u);
                    }
                    unsigned spins = 0;
                    while (true) {
                        // nearest tile with a running total: everything nearer contributes its own counts,
                        // everything farther is not needed (and not waited for)
                        unsigned tot[kWin];
                        int stop[kWin];
                        while (true) {
                            bool found = false, pending = false;
#pragma unroll
                            for (int w = 0; w < kWin; ++w) {
                                tot[w] = __ballot_sync(0xFFFFFFFFu, rec[w].w == 2u);
                                stop[w] = found ? -1 : (tot[w] ? (__ffs(tot[w]) - 1) : 32);
                                found |= tot[w] != 0u;
                                pending |= (lane <= stop[w]) && rec[w].w == 0u;
                            }
                            if (!__any_sync(0xFFFFFFFFu, pending)) break;
#pragma unroll
                            for (int w = 0; w < kWin; ++w) {
                                const int at = look - lane - 32 * w;
                                if (at >= 0 && rec[w].w == 0u) rec[w] = __ldcg(&desc[at]);
                            }
                            const bool bail = (++spins > kLookbackSpinLimit) || *reinterpret_cast<volatile int*>(&sy.abort) ||
                                              (*reinterpret_cast<volatile int*>(status) == MLMC_ERR_TIMEOUT);
                            if (__any_sync(0xFFFFFFFFu, bail)) {  // warp-uniform exit
                                ok = false;
                                break;
                            }
                        }
                        if (!ok) break;
                        uint32_t sC = 0, sA = 0, sB = 0;
                        unsigned any_tot = 0;
#pragma unroll
                        for (int w = 0; w < kWin; ++w) {
                            const bool use = lane <= stop[w];
                            sC += use ? rec[w].x : 0u;
                            sA += use ? rec[w].y : 0u;
                            sB += use ? rec[w].z : 0u;
                            any_tot |= tot[w];
                        }
                        pC += __reduce_add_sync(0xFFFFFFFFu, sC);
                        pA += __reduce_add_sync(0xFFFFFFFFu, sA);
                        pB += __reduce_add_sync(0xFFFFFFFFu, sB);
                        if (any_tot) break;
                        look -= 32 * kWin;
#pragma unroll
                        for (int w = 0; w < kWin; ++w) {
                            const int at = look - lane - 32 * w;
                            rec[w] = (at >= 0) ? __ldcg(&desc[at]) : make_uint4(0u, 0u, 0u, 2u);
                        }
                    }
                    if (lane == 0) put_record(&desc[t], pC + aggC, pA + aggA, pB + aggB, 2u);  // also after a give-up
                    if (!ok) {
                        set_status(status, MLMC_ERR_TIMEOUT);
                        worker_err[m] = MLMC_ERR_TIMEOUT;
                    }
                }
                // self-check on the worker's last tile: the band has exactly k_l - k_{l-1} entries
                if (lane == 0 && ok && t == tiles_per_worker - 1 &&
                    band_prefix(pC + aggC, pA + aggA, pB + aggB, e.ra, e.rb) != e.expect)
                    set_status(status, MLMC_ERR_INTERNAL);
            }
            if (lane == 0) {
                sh_pre[slot][0] = pC; sh_pre[slot][1] = pA; sh_pre[slot][2] = pB;
                sh_pre[slot][3] = (e.enabled && ok) ? 1u : 0u;
                *reinterpret_cast<volatile unsigned*>(&sy.ready[slot]) = j + 1u;
            }
        }
    }
    if (*reinterpret_cast<volatile int*>(&sy.abort)) set_status(status, MLMC_ERR_TIMEOUT);
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

}  // namespace

int configure_emit_kernels() {
    const int smem = kEmitStages * kEmitTile * (int)sizeof(uint32_t) + kEmitMaxWorkers * (int)sizeof(EmitParams);  // ring + band parameters
    if (cudaFuncSetAttribute(emit_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return MLMC_ERR_CUDA;
    if (cudaFuncSetAttribute(emit_kernel<bf16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return MLMC_OK;
}

void launch_emit(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const mlmc_topk_msgs& out,
                 cudaStream_t s) {
    const int per_word = (dtype == MLMC_BF16) ? 2 : 1;
    const int64_t words = (d + per_word - 1) / per_word;
    const int tpw = (int)((words + kEmitTile - 1) / kEmitTile);
    const unsigned total = (unsigned)tpw * (unsigned)M;
    cudaMemsetAsync(ws.tile_desc, 0, (size_t)total * sizeof(uint4), s);
    cudaMemsetAsync(ws.tile_counter, 0, sizeof(unsigned), s);
    unsigned grid = (unsigned)(ws.sm_count * kEmitBlocksPerSM);  // persistent blocks
    if (grid > total) grid = total;
    const size_t smem = (size_t)kEmitStages * kEmitTile * sizeof(uint32_t) + (size_t)M * sizeof(EmitParams);
    LaunchScope t(ws, K_EMIT, s);
    if (dtype == MLMC_BF16)
        emit_kernel<bf16_t><<<grid, kEmitThreads, smem, s>>>(static_cast<const bf16_t*>(g), d, ld, tpw, total, M, ws.emit,
                                                           ws.tile_desc, ws.tile_counter, out.idx, out.val, out.capacity,
                                                           ws.status, ws.worker_err);
    else
        emit_kernel<float><<<grid, kEmitThreads, smem, s>>>(static_cast<const float*>(g), d, ld, tpw, total, M, ws.emit,
                                                          ws.tile_desc, ws.tile_counter, out.idx, out.val, out.capacity,
                                                          ws.status, ws.worker_err);
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
    aggregate_topk_kernel<<<grid, 256, 2 * M * sizeof(uint32_t), s>>>(msgs.idx, msgs.val, msgs.capacity, M, d, ntiles,
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
uint32_t* g_static_offsets_addr[kMaxDevices];  // device address of the array on each device, 0 = not looked up yet
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
    if (!g_static_offsets_addr[dev]) {
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
        g_static_offsets_addr[dev] = p;
    }
    uint32_t* offsets = g_static_offsets_addr[dev];
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
