// MLMC with the floating-point bit-wise compressor (Sec. 2.2 "Floating-point compressors", App. B).
//
// An entry is e = (-1)^S 2^(E - bias) (1 + sum_j m_j 2^-j).  C^l keeps sign, exponent and the first mb_l mantissa
// digits; the residual C^l - C^{l-1} is the field of digits mb_{l-1}+1 .. mb_l, worth f 2^-mb_l 2^(E - bias).  Sign
// and exponent are sent with every message (App. B counts 1 + exponent + 1 bits per entry), and they are the base
// g^0 = sign 2^(E - bias) of the estimate g^0 + (1/p^l)(C^l - C^{l-1}).  The level draw does not depend on the data
// (App. B's lemma gives fixed probabilities), so one sweep over the gradient writes the whole message.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kFloatThreads = 256;

struct MantissaSchedule {
    int L;
    int lo[kMaxLevels];  // mb_{l-1}
    int hi[kMaxLevels];  // mb_l
};

MantissaSchedule make_mantissa_schedule(const int32_t* mb, int L) {
    MantissaSchedule sc = {};
    sc.L = L;
    for (int l = 0; l < L; ++l) {
        sc.lo[l] = l ? mb[l - 1] : 0;
        sc.hi[l] = mb[l];
    }
    return sc;
}

// Level and header of every worker.
__global__ void float_draw_kernel(const double* __restrict__ p_fixed, MantissaSchedule sc, uint64_t seed, uint64_t step,
                                  int M, int w_max, double* u_dev, int32_t* bit_level, int32_t* out_level,
                                  double* out_p_sel, int* status, int* worker_err) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    const double u = counter_uniform(seed, step, (uint64_t)m);
    u_dev[m] = u;
    int level = draw_from_probs(p_fixed, sc.L, u);
    const double p = p_fixed[level];
    if (sc.hi[level] - sc.lo[level] > w_max) {
        worker_err[m] = MLMC_ERR_CAPACITY;
        set_status(status, MLMC_ERR_CAPACITY);
        level = -1;
    }
    bit_level[m] = level;
    out_level[m] = level;
    out_p_sel[m] = level >= 0 ? p : 0.0;
}

// Every warp turns 1024 consecutive entries into 32 words of the sign plane and of each mantissa plane (one warp
// ballot per row of 32 entries and plane), and into 1024 exponent bytes, which leave through a shared-memory
// transpose as 32 consecutive bytes per lane.  All 32 rows of a group are requested before the first is used.
template <typename T>
__global__ void __launch_bounds__(kFloatThreads)
float_pack_kernel(const T* __restrict__ g, int64_t d, int64_t ld, MantissaSchedule sc,
                  const int32_t* __restrict__ bit_level, uint8_t* __restrict__ expo, uint32_t* __restrict__ planes,
                  int w_max, int64_t words, int32_t* out_level, int* status, int* worker_err) {
    __shared__ __align__(16) uint8_t sh_expo[kFloatThreads / 32][1024];
    const int m = blockIdx.y;
    const int level = bit_level[m];
    if (level < 0) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lo = sc.lo[level], w = sc.hi[level] - lo;
    const T* row = g + (int64_t)m * ld;
    uint32_t* out = planes + (int64_t)m * (1 + w_max) * words;
    uint8_t* ex = expo + (int64_t)m * words * 32;
    const int64_t ngroups = (words + 31) / 32;
    const int64_t stride = (int64_t)gridDim.x * (kFloatThreads / 32);
    bool bad = false;
    for (int64_t grp = (int64_t)blockIdx.x * (kFloatThreads / 32) + warp; grp < ngroups; grp += stride) {
        const int64_t e0 = grp * 1024;
        uint32_t x[32];  // fp32 encodings of this lane's entry of every row (entries past d read as +0)
        if (e0 + 1024 <= d) {
#pragma unroll
            for (int s = 0; s < 32; ++s) {
                if constexpr (sizeof(T) == 4)
                    x[s] = __ldg(reinterpret_cast<const uint32_t*>(row) + e0 + s * 32 + lane);
                else
                    x[s] = (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(row) + e0 + s * 32 + lane) << 16;
            }
        } else {
#pragma unroll
            for (int s = 0; s < 32; ++s) {
                const int64_t i = e0 + s * 32 + lane;
                x[s] = 0u;
                if (i < d) {
                    if constexpr (sizeof(T) == 4)
                        x[s] = reinterpret_cast<const uint32_t*>(row)[i];
                    else
                        x[s] = (uint32_t)reinterpret_cast<const uint16_t*>(row)[i] << 16;
                }
            }
        }
        const int64_t word = grp * 32 + lane;
        uint32_t sign_w = 0;
#pragma unroll
        for (int s = 0; s < 32; ++s) {
            const uint32_t bs = __ballot_sync(0xFFFFFFFFu, (int)x[s] < 0);
            if (lane == s) sign_w = bs;
            const uint32_t E = (x[s] >> 23) & 0xFFu;
            bad |= E == 0xFFu;
            sh_expo[warp][s * 32 + lane] = (uint8_t)E;
        }
        if (word < words) out[word] = sign_w;
        for (int j = 1; j <= w; ++j) {
            const int bit = 23 - (lo + j);  // mantissa digit lo + j of the fp32 encoding
            uint32_t mine = 0;
#pragma unroll
            for (int s = 0; s < 32; ++s) {
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, (x[s] >> bit) & 1u);
                if (lane == s) mine = b;
            }
            if (word < words) out[(int64_t)j * words + word] = mine;
        }
        __syncwarp();
        if (word < words) {  // the 32 exponent bytes of word `word`: rows are contiguous in the shared-memory matrix
            const uint4 a = reinterpret_cast<const uint4*>(&sh_expo[warp][lane * 32])[0];
            const uint4 b = reinterpret_cast<const uint4*>(&sh_expo[warp][lane * 32])[1];
            reinterpret_cast<uint4*>(ex + word * 32)[0] = a;
            reinterpret_cast<uint4*>(ex + word * 32)[1] = b;
        }
        __syncwarp();
    }
    if (bad) {  // NaN or Inf: the worker's message is void
        worker_err[m] = MLMC_ERR_NONFINITE;
        set_status(status, MLMC_ERR_NONFINITE);
        out_level[m] = -1;
    }
}

// Server average: thread = one word (32 entries); terms are added in worker order in fp32.
__global__ void __launch_bounds__(kFloatThreads)
aggregate_float_kernel(const uint8_t* __restrict__ expo, const uint32_t* __restrict__ planes,
                       const int32_t* __restrict__ level, const double* __restrict__ p_sel, MantissaSchedule sc,
                       int w_max, int64_t words, int M, int64_t d, float* __restrict__ out) {
    __shared__ float sh_out[kFloatThreads / 32][32][33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float inv_M = 1.0f / (float)M;
    const int64_t nblk = (words + kFloatThreads - 1) / kFloatThreads;
    for (int64_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
        const int64_t word = blk * kFloatThreads + threadIdx.x;
        float acc[32];
#pragma unroll
        for (int t = 0; t < 32; ++t) acc[t] = 0.0f;
        if (word < words) {
            for (int m = 0; m < M; ++m) {  // fixed worker order
                const int lv = level[m];
                if (lv < 0) continue;
                const int w = sc.hi[lv] - sc.lo[lv];
                const float c = (float)(ldexp(1.0, -sc.hi[lv]) / p_sel[m]);  // 2^-mb_l / p_l
                const uint32_t* pm = planes + (int64_t)m * (1 + w_max) * words;
                const uint8_t* em = expo + ((int64_t)m * words + word) * 32;
                const uint32_t sgn = pm[word];
                const uint4 ea = reinterpret_cast<const uint4*>(em)[0], eb = reinterpret_cast<const uint4*>(em)[1];
                const uint32_t eb4[8] = {ea.x, ea.y, ea.z, ea.w, eb.x, eb.y, eb.z, eb.w};
                uint32_t f[32];
#pragma unroll
                for (int t = 0; t < 32; ++t) f[t] = 0u;
                for (int j = 1; j <= w; ++j) {
                    const uint32_t pw = pm[(int64_t)j * words + word];
#pragma unroll
                    for (int t = 0; t < 32; ++t) f[t] = (f[t] << 1) | ((pw >> t) & 1u);
                }
#pragma unroll
                for (int t = 0; t < 32; ++t) {
                    const uint32_t E = (eb4[t >> 2] >> (8 * (t & 3))) & 0xFFu;
                    // exponent field 0: no leading one, and the scale of exponent field 1
                    const float base = __uint_as_float(E << 23);                   // 2^(E - 127), or 0
                    const float scale = __uint_as_float(max(E, 1u) << 23);         // 2^(max(E, 1) - 127)
                    const float ff = __uint_as_float(0x4B000000u | f[t]) - 8388608.0f;  // exact integer-to-float
                    const float v = fmaf(ff * c, scale, base);  // the power of two last: ff c is a normal number
                    acc[t] += __uint_as_float(__float_as_uint(v) ^ (((sgn >> t) & 1u) << 31));
                }
            }
        }
#pragma unroll
        for (int t = 0; t < 32; ++t) sh_out[warp][lane][t] = acc[t] * inv_M;
        __syncwarp();
        const int64_t wbase = blk * kFloatThreads + warp * 32;
#pragma unroll 4
        for (int r = 0; r < 32; ++r) {
            const int64_t i = (wbase + r) * 32 + lane;
            if (i < d) out[i] = sh_out[warp][r][lane];
        }
        __syncwarp();
    }
}

}  // namespace

void launch_compress_floatbits(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* mb,
                               int L, uint64_t seed, uint64_t step, const mlmc_float_msgs& out, cudaStream_t s) {
    const MantissaSchedule sc = make_mantissa_schedule(mb, L);
    {
        LaunchScope t(ws, K_FLOAT_DRAW, s);
        float_draw_kernel<<<(M + 127) / 128, 128, 0, s>>>(ws.p_fixed, sc, seed, step, M, out.w_max, ws.u_dev, ws.bit_level,
                                                          out.level, out.p_sel, ws.status, ws.worker_err);
    }
    const int64_t words = (d + 31) / 32;
    const int64_t ngroups = (words + 31) / 32;
    const int64_t by_work = (ngroups + (kFloatThreads / 32) - 1) / (kFloatThreads / 32);
    int64_t nb = ((int64_t)ws.sm_count * 4) / M;  // whole waves of the blocks that fit an SM, rounded down
    if (nb > by_work) nb = by_work;
    if (nb < 1) nb = 1;
    LaunchScope t(ws, K_FLOAT_PACK, s);
    if (dtype == MLMC_BF16)
        float_pack_kernel<bf16_t><<<dim3((unsigned)nb, M), kFloatThreads, 0, s>>>(
            static_cast<const bf16_t*>(g), d, ld, sc, ws.bit_level, out.expo, out.planes, out.w_max, words, out.level,
            ws.status, ws.worker_err);
    else
        float_pack_kernel<float><<<dim3((unsigned)nb, M), kFloatThreads, 0, s>>>(
            static_cast<const float*>(g), d, ld, sc, ws.bit_level, out.expo, out.planes, out.w_max, words, out.level,
            ws.status, ws.worker_err);
}

void launch_aggregate_floatbits(Workspace& ws, const mlmc_float_msgs& msgs, const int32_t* mb, int L, int M, int64_t d,
                                float* out, cudaStream_t s) {
    const MantissaSchedule sc = make_mantissa_schedule(mb, L);
    const int64_t words = (d + 31) / 32;
    int64_t nb = (words + kFloatThreads - 1) / kFloatThreads;
    const int64_t cap = (int64_t)ws.sm_count * 8;
    if (nb > cap) nb = cap;
    LaunchScope t(ws, K_AGG_FLOAT, s);
    aggregate_float_kernel<<<(unsigned)nb, kFloatThreads, 0, s>>>(msgs.expo, msgs.planes, msgs.level, msgs.p_sel, sc,
                                                                  msgs.w_max, words, M, d, out);
}

}  // namespace mlmc
