// Band emission (ordered stream compaction) and the server-side average for MLMC-Top-k.
//
// emit: one sweep over every worker's gradient writes the band of the drawn level,
//   { i : k_{l-1} < rank(i) <= k_l },  as (i, g_i / p_l) in ascending i  (Eq. 5 with g^0 = 0; Alg. 2 "Send").
// Membership is decided from the two thresholds (Ta, ra), (Tb, rb) of the band; equal-key elements
// are admitted by their index-ordered rank, so the running counts
//   D  = #{ Tb < key <= Ta },  Ea = #{ key == Ta },  Eb = #{ key == Tb }
// are carried across tiles with a decoupled look-back (tiles are numbered by a ticket counter, so
// every predecessor of a running tile has already started; every wait is bounded).
//
// aggregate: the dense mean (1/M) sum_m g~_m (Alg. 2 "Server aggregates") tiled over the index
// space; because every message is index-sorted, a tile's entries are one contiguous range per
// worker; they are added into a shared-memory tile in worker order and the tile is written once.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr unsigned kSpinLimit = 1u << 22;  // polls before a look-back gives up (each poll is a global load)

// Look-back record of one tile: {D, Ea, Eb, state}, state 0 = not yet, 1 = the tile's own counts,
// 2 = running totals up to and including the tile.  A record is written and read as one 16-byte
// access, so counts and state always belong together.
__device__ __forceinline__ void put_record(uint4* rec, uint32_t D, uint32_t Ea, uint32_t Eb, uint32_t state) {
    __stcg(rec, make_uint4(D, Ea, Eb, state));
}

__device__ __forceinline__ uint32_t warp_sum(uint32_t x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    return x;
}

// One block per tile of kEmitTile consecutive entries of one worker (blockIdx.y).  Tiles are numbered by
// a per-worker ticket taken when the block starts, so every lower-numbered tile is already running and
// will publish its counts without waiting for anyone.
template <typename T>
__global__ void __launch_bounds__(kEmitThreads, 10)
emit_kernel(const T* __restrict__ g, int64_t d, int64_t ld, int tiles_per_worker,
            const EmitParams* __restrict__ emit, uint4* tile_desc, unsigned* tile_counter,
            uint32_t* __restrict__ idx_out, float* __restrict__ val_out, int64_t capacity, int* status,
            int* worker_err) {
    using Tr = ElemTraits<T>;
    constexpr int V = Tr::kVec;
    constexpr int NV = kEmitItems / V;
    constexpr int kWarps = kEmitThreads / 32;
    __shared__ unsigned sh_ticket;
    __shared__ unsigned long long sh_warp[kWarps];
    __shared__ uint32_t sh_prefix[4];  // D, Ea, Eb, ok
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m = blockIdx.y;
    const EmitParams e = emit[m];
    if (!e.enabled) return;
    if (threadIdx.x == 0) sh_ticket = atomicAdd(&tile_counter[m], 1u);
    __syncthreads();
    const int t = (int)sh_ticket;
    uint4* desc = tile_desc + (int64_t)m * tiles_per_worker;

    // ---- load this thread's 16 consecutive elements
    const T* row = g + (int64_t)m * ld;
    const int64_t i0 = (int64_t)t * kEmitTile + (int64_t)threadIdx.x * kEmitItems;
    uint32_t bits[kEmitItems];
    uint32_t valid = 0;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const int64_t base = i0 + j * V;
        if (base + V <= d) {
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(row + base));
            if constexpr (V == 4) {
                bits[j * 4 + 0] = q.x; bits[j * 4 + 1] = q.y; bits[j * 4 + 2] = q.z; bits[j * 4 + 3] = q.w;
            } else {
                bits[j * 8 + 0] = q.x & 0xFFFFu; bits[j * 8 + 1] = q.x >> 16;
                bits[j * 8 + 2] = q.y & 0xFFFFu; bits[j * 8 + 3] = q.y >> 16;
                bits[j * 8 + 4] = q.z & 0xFFFFu; bits[j * 8 + 5] = q.z >> 16;
                bits[j * 8 + 6] = q.w & 0xFFFFu; bits[j * 8 + 7] = q.w >> 16;
            }
            valid |= ((1u << V) - 1u) << (j * V);
        } else {
#pragma unroll
            for (int c = 0; c < V; ++c) {
                bits[j * V + c] = 0;
                if (base + c < d) {
                    if constexpr (V == 4)
                        bits[j * V + c] = reinterpret_cast<const uint32_t*>(row)[base + c];
                    else
                        bits[j * V + c] = reinterpret_cast<const uint16_t*>(row)[base + c];
                    valid |= 1u << (j * V + c);
                }
            }
        }
    }

    // ---- local counts, packed 21 bits each: D | Ea << 21 | Eb << 42
    unsigned long long pack = 0;
#pragma unroll
    for (int i = 0; i < kEmitItems; ++i) {
        const uint32_t key = Tr::key(bits[i]);
        const bool ok = (valid >> i) & 1u;
        const unsigned long long dD = (ok && key > e.Tb && key <= e.Ta) ? 1ull : 0ull;
        const unsigned long long dA = (ok && key == e.Ta) ? 1ull : 0ull;
        const unsigned long long dB = (ok && key == e.Tb) ? 1ull : 0ull;
        pack += dD | (dA << 21) | (dB << 42);
    }
    unsigned long long inc = pack;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31) sh_warp[warp] = inc;
    __syncthreads();
    unsigned long long warp_off = 0, block_total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const unsigned long long s = sh_warp[w];
        if (w < warp) warp_off += s;
        block_total += s;
    }
    const unsigned long long excl = inc - pack + warp_off;
    const uint32_t aggD = (uint32_t)(block_total & 0x1FFFFFu);
    const uint32_t aggA = (uint32_t)((block_total >> 21) & 0x1FFFFFu);
    const uint32_t aggB = (uint32_t)((block_total >> 42) & 0x1FFFFFu);

    // ---- decoupled look-back over this worker's earlier tiles (warp 0)
    if (warp == 0) {
        uint32_t pD = 0, pA = 0, pB = 0;
        bool ok = true;
        if (t > 0) {
            if (lane == 0) put_record(&desc[t], aggD, aggA, aggB, 1u);
            int look = t - 1;
            unsigned spins = 0;
            while (true) {
                const int at = look - lane;
                // positions before the worker's first tile count as an empty running total
                uint4 rec = (at >= 0) ? __ldcg(&desc[at]) : make_uint4(0u, 0u, 0u, 2u);
                while (!__all_sync(0xFFFFFFFFu, rec.w != 0u)) {
                    if (at >= 0 && rec.w == 0u) rec = __ldcg(&desc[at]);
                    const bool bail = (++spins > kSpinLimit) ||
                                      (*reinterpret_cast<volatile int*>(status) == MLMC_ERR_TIMEOUT);
                    if (__any_sync(0xFFFFFFFFu, bail)) {  // warp-uniform exit
                        ok = false;
                        break;
                    }
                }
                if (!ok) break;
                const unsigned has_total = __ballot_sync(0xFFFFFFFFu, rec.w == 2u);
                const int stop = has_total ? (__ffs(has_total) - 1) : 32;  // nearest tile with a running total
                const bool use = lane <= stop;
                pD += warp_sum(use ? rec.x : 0u);
                pA += warp_sum(use ? rec.y : 0u);
                pB += warp_sum(use ? rec.z : 0u);
                if (has_total) break;
                look -= 32;
            }
            if (!ok) {
                set_status(status, MLMC_ERR_TIMEOUT);
                worker_err[m] = MLMC_ERR_TIMEOUT;
            }
        }
        if (lane == 0) {
            put_record(&desc[t], pD + aggD, pA + aggA, pB + aggB, 2u);  // also after a give-up, so successors move on
            sh_prefix[0] = pD; sh_prefix[1] = pA; sh_prefix[2] = pB; sh_prefix[3] = ok ? 1u : 0u;
        }
    }
    __syncthreads();
    const bool ok = sh_prefix[3] != 0;
    uint32_t rD = sh_prefix[0] + (uint32_t)(excl & 0x1FFFFFu);
    uint32_t rA = sh_prefix[1] + (uint32_t)((excl >> 21) & 0x1FFFFFu);
    uint32_t rB = sh_prefix[2] + (uint32_t)((excl >> 42) & 0x1FFFFFu);

    // ---- self-check on the worker's last tile: the band has exactly k_l - k_{l-1} entries
    if (t == tiles_per_worker - 1 && threadIdx.x == 0 && ok) {
        const uint32_t tD = sh_prefix[0] + aggD, tA = sh_prefix[1] + aggA, tB = sh_prefix[2] + aggB;
        const uint32_t total = tD + min(tB, e.rb) - min(tA, e.ra);
        if (total != e.expect) set_status(status, MLMC_ERR_INTERNAL);
    }

    // ---- write the band entries at their global positions
    if (ok && (aggD | aggA | aggB)) {
        uint32_t* idx_w = idx_out + (int64_t)m * capacity;
        float* val_w = val_out + (int64_t)m * capacity;
#pragma unroll
        for (int i = 0; i < kEmitItems; ++i) {
            const uint32_t key = Tr::key(bits[i]);
            const bool okv = (valid >> i) & 1u;
            const bool eqA = okv && key == e.Ta, eqB = okv && key == e.Tb;
            const bool insA = okv && (key > e.Ta || (eqA && rA < e.ra));   // tie rank rA + 1 <= ra
            const bool insB = okv && (key > e.Tb || (eqB && rB < e.rb));
            if (insB && !insA) {
                const uint32_t pos = rD + min(rB, e.rb) - min(rA, e.ra);
                if ((int64_t)pos < capacity) {
                    idx_w[pos] = (uint32_t)(i0 + i);
                    val_w[pos] = (float)((double)Tr::value(bits[i]) * e.inv_p);
                }
            }
            rD += (okv && key > e.Tb && key <= e.Ta) ? 1u : 0u;
            rA += eqA ? 1u : 0u;
            rB += eqB ? 1u : 0u;
        }
    }
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

__global__ void __launch_bounds__(256)
aggregate_topk_kernel(const uint32_t* __restrict__ idx, const float* __restrict__ val, int64_t capacity, int M,
                      int64_t d, int ntiles, const uint32_t* __restrict__ offsets, float* __restrict__ out) {
    __shared__ float acc[kAggTile];
    const float fM = (float)M;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t base = (int64_t)t * kAggTile;
        for (int i = threadIdx.x; i < kAggTile; i += blockDim.x) acc[i] = 0.0f;
        __syncthreads();
        for (int m = 0; m < M; ++m) {  // fixed worker order: reproducible fp32 sums
            const uint32_t o0 = offsets[(int64_t)m * (ntiles + 1) + t];
            const uint32_t o1 = offsets[(int64_t)m * (ntiles + 1) + t + 1];
            if (o1 > o0) {
                const uint32_t* a = idx + (int64_t)m * capacity;
                const float* v = val + (int64_t)m * capacity;
                for (uint32_t j = o0 + threadIdx.x; j < o1; j += blockDim.x)
                    acc[a[j] - (uint32_t)base] += v[j];  // indices are unique within a worker
                __syncthreads();
            }
        }
        for (int i = threadIdx.x; i < kAggTile; i += blockDim.x)
            if (base + i < d) out[base + i] = acc[i] / fM;
        __syncthreads();
    }
}

}  // namespace

void launch_emit(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const mlmc_topk_msgs& out,
                 cudaStream_t s) {
    const int tpw = (int)((d + kEmitTile - 1) / kEmitTile);
    cudaMemsetAsync(ws.tile_desc, 0, (size_t)tpw * M * sizeof(uint4), s);
    cudaMemsetAsync(ws.tile_counter, 0, sizeof(unsigned) * M, s);
    LaunchScope t(ws, K_EMIT, s);
    if (dtype == MLMC_BF16)
        emit_kernel<bf16_t><<<dim3(tpw, M), kEmitThreads, 0, s>>>(static_cast<const bf16_t*>(g), d, ld, tpw, ws.emit,
                                                                 ws.tile_desc, ws.tile_counter, out.idx, out.val,
                                                                 out.capacity, ws.status, ws.worker_err);
    else
        emit_kernel<float><<<dim3(tpw, M), kEmitThreads, 0, s>>>(static_cast<const float*>(g), d, ld, tpw, ws.emit,
                                                                ws.tile_desc, ws.tile_counter, out.idx, out.val,
                                                                out.capacity, ws.status, ws.worker_err);
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
    aggregate_topk_kernel<<<grid, 256, 0, s>>>(msgs.idx, msgs.val, msgs.capacity, M, d, ntiles, ws.agg_offsets, out);
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
    if (M < 1 || d < 1 || d >= (int64_t(1) << 32) || msgs->capacity < 0) return MLMC_ERR_ARG;
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
    aggregate_topk_kernel<<<(unsigned)grid, 256, 0, s>>>(msgs->idx, msgs->val, msgs->capacity, M, d, (int)ntiles,
                                                         offsets, out);
    return cudaGetLastError() == cudaSuccess ? MLMC_OK : MLMC_ERR_CUDA;
}
