// MLMC with the fixed-point bit-wise compressor (Sec. 3.1).
//
// Entries are divided by the largest magnitude of the worker's gradient and written as a sign plus
// B fractional bits (Eq. 6 with B = b_{L-1} <= 23 instead of 63, since the input is fp32/bf16):
//   e = fl32(|g| / gmax),  q = min(floor(e 2^B), 2^B - 1).
// Level l keeps the top b_l bits of q; the residual C^l - C^{l-1} is the field
//   f_l = (q >> (B - b_l)) & (2^{w_l} - 1),  w_l = b_l - b_{l-1},  worth  sign f_l 2^{-b_l} gmax,
// sent as one sign plane and w_l magnitude planes.  Adaptive probabilities (Lemma 3.4) use the exact
// integer field energies S_l = sum_i f_l^2:  Delta_l = gmax 2^{-b_l} sqrt(S_l).
#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kBitThreads = 256;

struct BitSchedule {
    int L;
    int B;
    int shift[kMaxLevels];      // B - b_l
    uint32_t mask[kMaxLevels];  // 2^{w_l} - 1
    int width[kMaxLevels];      // w_l
    int bits[kMaxLevels];       // b_l
};

// The code q = min(trunc(fl32(|g| / gmax) * 2^B), 2^B - 1) with the IEEE-rounded fp32 quotient, for a fixed
// divisor.  The quotient is formed in fp64 as |g| * (1 / gmax) and rounded to fp32 once: a quotient of two
// 24-bit significands is never closer than 2^-49 (relative) to the midpoint of two fp32 numbers, the fp64
// product is within 2^-52 of it, so this rounding is the same as that of the fp32 division.
struct Quantiser {
    double inv_scaled;  // fl64(1 / gmax) * 2^B
    uint32_t qmax;      // 2^B - 1
    bool widen_by_bits;  // gmax >= 2^-100: an fp32 operand below the normal range cannot reach q = 1, so its
                         // fp64 image may be built from the bit pattern as if it were normal
    __device__ __forceinline__ Quantiser(float g, int B) {
        inv_scaled = g > 0.0f ? ldexp(1.0 / (double)g, B) : 0.0;
        qmax = (1u << B) - 1u;
        widen_by_bits = g >= 0x1.0p-100f;
    }
    __device__ __forceinline__ uint32_t code(uint32_t mag_bits /* sign bit cleared */) const {
        double x;
        if (widen_by_bits)
            x = __hiloint2double((int)((mag_bits >> 3) + 0x38000000u), (int)(mag_bits << 29));
        else
            x = (double)__uint_as_float(mag_bits);
        // fl32(|g| / gmax) * 2^B in one rounding: scaling by a power of two commutes with both roundings (a
        // quotient so small that its fp32 image would be subnormal has the code 0 either way)
        const float scaled = (float)(x * inv_scaled);
        return min(__float2uint_rz(scaled), qmax);  // truncation: the lower bits are discarded
    }
};

// ---- per-worker max |g| as an integer max over magnitude keys; flags NaN / Inf
template <typename T>
__global__ void __launch_bounds__(kSweepThreads)
absmax_kernel(const T* __restrict__ g, int64_t d, int64_t ld, uint32_t* gmax_bits, int* status, int* worker_err) {
    using Tr = ElemTraits<T>;
    __shared__ uint32_t sh_max[kSweepThreads / 32];
    const int m = blockIdx.y;
    const T* row = g + (int64_t)m * ld;
    int64_t v0, v1;
    block_vector_range(d, Tr::kVec, blockIdx.x, gridDim.x, &v0, &v1);
    uint32_t mx = 0;
    // four 16-byte loads per thread are in flight before any is used
    constexpr int kBatch = 4;
    const int64_t full_end = min(v1, d / Tr::kVec);  // vectors wholly inside the row
    int64_t v = v0 + threadIdx.x;
    for (; v + (int64_t)(kBatch - 1) * blockDim.x < full_end; v += (int64_t)kBatch * blockDim.x) {
        uint4 q[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) q[j] = __ldg(reinterpret_cast<const uint4*>(row) + v + (int64_t)j * blockDim.x);
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            if constexpr (Tr::kVec == 4) {
                mx = max(max(mx, q[j].x & 0x7FFFFFFFu), max(q[j].y & 0x7FFFFFFFu, max(q[j].z & 0x7FFFFFFFu, q[j].w & 0x7FFFFFFFu)));
            } else {
                // both halves at once: the low halves after masking, the high halves shifted down
                const uint32_t a = max(max(q[j].x & 0x7FFFu, q[j].y & 0x7FFFu), max(q[j].z & 0x7FFFu, q[j].w & 0x7FFFu));
                const uint32_t b = max(max((q[j].x >> 16) & 0x7FFFu, (q[j].y >> 16) & 0x7FFFu),
                                       max((q[j].z >> 16) & 0x7FFFu, (q[j].w >> 16) & 0x7FFFu));
                mx = max(mx, max(a, b));
            }
        }
    }
    for (; v < v1; v += blockDim.x)
        for_each_in_vector<T>(row, v, d, [&](int64_t, uint32_t bits) { mx = max(mx, Tr::key(bits)); });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    if ((threadIdx.x & 31) == 0) sh_max[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kSweepThreads / 32; ++w) mx = max(mx, sh_max[w]);
        if (mx >= Tr::kInfKey) {
            worker_err[m] = MLMC_ERR_NONFINITE;
            set_status(status, MLMC_ERR_NONFINITE);
        }
        const uint32_t as_f32 = (Tr::kVec == 8) ? (mx << 16) : mx;
        atomicMax(&gmax_bits[m], as_f32);
    }
}

// ---- adaptive only: exact field energies S_l = sum_i f_l^2 for every level in one sweep
// Acc = uint32_t when every field is at most 8 bits wide and a thread sees fewer than 2^16 entries (f^2 < 2^16,
// so the sum fits 32 bits), else unsigned long long.  Fields come from the prefix codes P_l = q >> (B - b_l):
// f_l = P_l - (P_{l-1} << w_l), one shift and one multiply-add per level.
template <typename T, int LMAX, typename Acc>
__global__ void __launch_bounds__(kSweepThreads)
bit_stats_kernel(const T* __restrict__ g, int64_t d, int64_t ld, const uint32_t* __restrict__ gmax_bits,
                 BitSchedule sc, unsigned long long* __restrict__ S_partial, int stat_ctas, const int* worker_err) {
    using Tr = ElemTraits<T>;
    __shared__ unsigned long long sh_red[kSweepThreads / 32];
    const int m = blockIdx.y;
    if (worker_err[m]) return;
    const float gmax = __uint_as_float(gmax_bits[m]);
    const Quantiser qz(gmax, sc.B);
    Acc acc[LMAX];
    int sh[LMAX];
    uint32_t neg_pow[LMAX];
#pragma unroll
    for (int l = 0; l < LMAX; ++l) {  // the schedule in registers; levels past L get shift 0 and width 0: their field is q - q = 0
        acc[l] = 0;
        sh[l] = (l < sc.L) ? sc.shift[l] : 0;
        neg_pow[l] = 0u - (1u << ((l < sc.L) ? sc.width[l] : 0));
    }
    if (gmax > 0.0f) {
        const T* row = g + (int64_t)m * ld;
        int64_t v0, v1;
        block_vector_range(d, Tr::kVec, blockIdx.x, gridDim.x, &v0, &v1);
        auto take = [&](uint32_t bits) {
            const uint32_t q = qz.code(__float_as_uint(Tr::value(bits)) & 0x7FFFFFFFu);
            uint32_t prev = 0;  // P_{l-1}
#pragma unroll
            for (int l = 0; l < LMAX; ++l) {
                const uint32_t P = q >> sh[l];
                const uint32_t f = prev * neg_pow[l] + P;
                acc[l] += (Acc)f * f;
                prev = P;
            }
        };
        // two 16-byte loads per thread are in flight before either is used
        constexpr int kBatch = 2;
        const int64_t full_end = min(v1, d / Tr::kVec);  // vectors wholly inside the row
        int64_t v = v0 + threadIdx.x;
        for (; v + (int64_t)(kBatch - 1) * blockDim.x < full_end; v += (int64_t)kBatch * blockDim.x) {
            uint4 qv[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) qv[j] = __ldg(reinterpret_cast<const uint4*>(row) + v + (int64_t)j * blockDim.x);
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                if constexpr (Tr::kVec == 4) {
                    take(qv[j].x); take(qv[j].y); take(qv[j].z); take(qv[j].w);
                } else {
                    take(qv[j].x & 0xFFFFu); take(qv[j].x >> 16); take(qv[j].y & 0xFFFFu); take(qv[j].y >> 16);
                    take(qv[j].z & 0xFFFFu); take(qv[j].z >> 16); take(qv[j].w & 0xFFFFu); take(qv[j].w >> 16);
                }
            }
        }
        for (; v < v1; v += blockDim.x) for_each_in_vector<T>(row, v, d, [&](int64_t, uint32_t bits) { take(bits); });
    }
#pragma unroll
    for (int l = 0; l < LMAX; ++l) {
        if (l >= sc.L) break;
        unsigned long long x = (unsigned long long)acc[l];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
        if ((threadIdx.x & 31) == 0) sh_red[threadIdx.x >> 5] = x;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long s = 0;
            for (int w = 0; w < kSweepThreads / 32; ++w) s += sh_red[w];
            S_partial[((int64_t)m * stat_ctas + blockIdx.x) * kMaxLevels + l] = s;
        }
        __syncthreads();
    }
}

__device__ int draw_level_bits(const double* p, int L, double u) {
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

// ---- probabilities, draw and message header of every worker (one warp per worker)
__global__ void bit_probs_draw_kernel(BitSchedule sc, const uint32_t* gmax_bits, const unsigned long long* S_partial,
                                      int n_partials, int stat_ctas, const double* p_fixed, int adaptive,
                                      int need_delta, uint64_t seed, uint64_t step, int M, double* p_all,
                                      double* delta_all, double* u_dev, int32_t* bit_level, float* out_gmax,
                                      int32_t* out_level, double* out_p_sel, int w_max, int want_msg, int* status,
                                      int* worker_err) {
    const int m = blockIdx.x;
    const int lane = threadIdx.x;
    if (m >= M) return;
    if (worker_err[m]) {
        if (lane == 0) {
            bit_level[m] = -1;
            if (want_msg) {
                out_level[m] = -1;
                out_p_sel[m] = 0.0;
                out_gmax[m] = 0.0f;
            }
        }
        return;
    }
    const float gmax = __uint_as_float(gmax_bits[m]);
    double p[kMaxLevels], delta[kMaxLevels];
    if (adaptive || need_delta) {
        for (int l = 0; l < sc.L; ++l) {
            // exact 128-bit sum of the per-block partials (lanes take every 32nd, integer adds: any order),
            // rounded once to fp64
            unsigned __int128 S = 0;
            for (int c = lane; c < n_partials; c += 32) S += S_partial[((int64_t)m * stat_ctas + c) * kMaxLevels + l];
            unsigned long long lo = (unsigned long long)S, hi = (unsigned long long)(S >> 64);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long lo2 = __shfl_xor_sync(0xFFFFFFFFu, lo, o), hi2 = __shfl_xor_sync(0xFFFFFFFFu, hi, o);
                const unsigned __int128 t = (((unsigned __int128)hi << 64) | lo) + (((unsigned __int128)hi2 << 64) | lo2);
                lo = (unsigned long long)t;
                hi = (unsigned long long)(t >> 64);
            }
            const double Sd = (double)hi * 0x1.0p64 + (double)lo;
            delta[l] = (double)gmax * ldexp(1.0, -sc.bits[l]) * sqrt(Sd);
        }
    }
    if (lane != 0) return;
    if (adaptive || need_delta)
        for (int l = 0; l < sc.L; ++l) delta_all[m * kMaxLevels + l] = delta[l];
    if (adaptive) {
        double s = 0.0;
        for (int l = 0; l < sc.L; ++l) s += delta[l];
        for (int l = 0; l < sc.L; ++l) p[l] = (s > 0.0) ? delta[l] / s : (l == 0 ? 1.0 : 0.0);
    } else {
        for (int l = 0; l < sc.L; ++l) p[l] = p_fixed[l];
    }
    for (int l = 0; l < sc.L; ++l) p_all[m * kMaxLevels + l] = p[l];
    const double u = counter_uniform(seed, step, (uint64_t)m);
    u_dev[m] = u;
    int level = draw_level_bits(p, sc.L, u);
    if (want_msg) {
        if (sc.width[level] > w_max) {
            worker_err[m] = MLMC_ERR_CAPACITY;
            set_status(status, MLMC_ERR_CAPACITY);
            level = -1;
        }
        out_level[m] = level;
        out_p_sel[m] = (level >= 0) ? p[level] : 0.0;
        out_gmax[m] = gmax;
    }
    bit_level[m] = level;
}

// ---- pack: every warp turns 1024 consecutive entries into 32 words of each plane.
// The entries of a group are staged in a two-slot shared-memory ring private to the warp: the next group's
// copy (cp.async) is in flight while the current group is coded and packed.
// WIDE = false serves the workers whose drawn level has a field of at most 8 bits, WIDE = true the others (each
// instance leaves the other's workers alone): the narrow path keeps no per-row state in registers, which the wide
// path's 32 codes per lane would otherwise force on it.
template <typename T, bool WIDE>
__global__ void __launch_bounds__(kBitThreads, WIDE ? 2 : 3)
bit_pack_kernel(const T* __restrict__ g, int64_t d, int64_t ld, const uint32_t* __restrict__ gmax_bits,
                BitSchedule sc, const int32_t* __restrict__ bit_level, uint32_t* __restrict__ planes, int w_max,
                int64_t words) {
    using Tr = ElemTraits<T>;
    constexpr int kGroup = 1024;
    constexpr int kGroupBytes = kGroup * (int)sizeof(T);
    extern __shared__ __align__(16) uint8_t sh_pack[];  // [warps][2][kGroupBytes], then [warps][1024] field bytes
    const int m = blockIdx.y;
    const int level = bit_level[m];
    if (level < 0) return;
    if ((sc.width[level] > 8) != WIDE) return;  // the other instance's worker
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps_per_block = kBitThreads / 32;
    const int64_t ngroups = (words + 31) / 32;  // groups of 32 words = 1024 entries
    const float gmax = __uint_as_float(gmax_bits[m]);
    const Quantiser qz(gmax, sc.B);
    const int shift = sc.shift[level];
    const uint32_t mask = sc.mask[level];
    const int w = sc.width[level];
    const T* row = g + (int64_t)m * ld;
    uint32_t* out = planes + (int64_t)m * (1 + w_max) * words;
    uint8_t* ring = sh_pack + warp * 2 * kGroupBytes;
    uint8_t* bytes = sh_pack + warps_per_block * 2 * kGroupBytes + warp * 1024;  // 32 rows x 32 field bytes
    auto fetch = [&](int64_t grp, int stage) {  // one commit per call
        if (grp < ngroups) {
            const int64_t e0 = grp * kGroup;
            uint8_t* dst = ring + stage * kGroupBytes;
            if (e0 + kGroup <= d) {
                const uint8_t* src = reinterpret_cast<const uint8_t*>(row + e0);
#pragma unroll
                for (int c = lane; c < kGroupBytes / 16; c += 32) cp_async_16(dst + c * 16, src + c * 16);
            } else {  // ragged last group: entries past d read as +0
                for (int i = lane; i < kGroup; i += 32) {
                    if constexpr (Tr::kVec == 4)
                        reinterpret_cast<uint32_t*>(dst)[i] = (e0 + i < d) ? reinterpret_cast<const uint32_t*>(row)[e0 + i] : 0u;
                    else
                        reinterpret_cast<uint16_t*>(dst)[i] = (e0 + i < d) ? reinterpret_cast<const uint16_t*>(row)[e0 + i] : (uint16_t)0;
                }
            }
        }
        cp_async_commit();
    };
    const int64_t stride = (int64_t)gridDim.x * warps_per_block;
    int64_t grp = (int64_t)blockIdx.x * warps_per_block + warp;
    // An entry below gmax 2^-b_l (1 - 2^-20) has fl32(|g| / gmax) < 2^-b_l, so its top b_l code bits and with them
    // the field of level l are zero.  A row of 32 entries that are all below that bound is not coded at all: in
    // a gradient with per-layer scales and a few outliers this is most rows of the high levels.
    const uint32_t zero_below = (gmax > 0.0f) ? __float_as_uint(gmax * ldexpf(1.0f - 0x1.0p-20f, -sc.bits[level])) : 0x7FFFFFFFu;
    fetch(grp, 0);
    for (int it = 0; grp < ngroups; grp += stride, ++it) {
        fetch(grp + stride, (it + 1) & 1);
        cp_async_wait<1>();  // this group has landed (the next one may still be in flight)
        __syncwarp();
        const uint8_t* buf = ring + (it & 1) * kGroupBytes;
        const int64_t word = grp * 32 + lane;
        auto entry_bits = [&](int s) -> uint32_t {
            uint32_t bits;
            if constexpr (Tr::kVec == 4)
                bits = reinterpret_cast<const uint32_t*>(buf)[s * 32 + lane];
            else
                bits = reinterpret_cast<const uint16_t*>(buf)[s * 32 + lane];
            return __float_as_uint(Tr::value(bits));
        };
        if constexpr (!WIDE) {
            // Fields of at most 8 bits go through a byte matrix in shared memory: lane L writes the field of each of
            // its 32 rows, then lane r gathers bit b of the 32 bytes of row r, four bytes per multiply
            // (((x >> b) & 0x01010101) * 0x01020408 puts the four bits side by side in bits 24..27).  This costs
            // a quarter of one ballot per row and plane.  The sign plane takes one ballot per row.
            uint32_t sign_w = 0;
            bool coded = false;  // warp-uniform: some row of the group was coded
#pragma unroll
            for (int s = 0; s < 32; ++s) {
                const uint32_t xb = entry_bits(s);
                const uint32_t bs = __ballot_sync(0xFFFFFFFFu, (int)xb < 0);
                if (lane == s) sign_w = bs;
                uint32_t f = 0;
                if (__any_sync(0xFFFFFFFFu, (xb & 0x7FFFFFFFu) >= zero_below)) {
                    f = (qz.code(xb & 0x7FFFFFFFu) >> shift) & mask;
                    coded = true;
                }
                bytes[s * 32 + lane] = (uint8_t)f;
            }
            __syncwarp();
            if (word < words) out[word] = sign_w;
            if (coded) {
                const uint4 lo = reinterpret_cast<const uint4*>(bytes + lane * 32)[0];
                const uint4 hi = reinterpret_cast<const uint4*>(bytes + lane * 32)[1];
                const uint32_t x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                for (int j = 1; j <= w; ++j) {
                    const int bit = w - j;
                    uint32_t pw = 0;
#pragma unroll
                    for (int c = 0; c < 8; ++c) pw |= ((((x[c] >> bit) & 0x01010101u) * 0x01020408u) >> 24 & 0xFu) << (4 * c);
                    if (word < words) out[(int64_t)j * words + word] = pw;
                }
            } else if (word < words) {  // every field of the group is zero
                for (int j = 1; j <= w; ++j) out[(int64_t)j * words + word] = 0u;
            }
        } else {
            uint32_t code[32];  // bit 31 = sign, low bits = field
#pragma unroll
            for (int s = 0; s < 32; ++s) {
                const uint32_t xb = entry_bits(s);
                code[s] = xb & 0x80000000u;
                if (__any_sync(0xFFFFFFFFu, (xb & 0x7FFFFFFFu) >= zero_below))
                    code[s] |= (qz.code(xb & 0x7FFFFFFFu) >> shift) & mask;
            }
            for (int j = 0; j <= w; ++j) {
                const int bit = (j == 0) ? 31 : (w - j);
                uint32_t mine = 0;
#pragma unroll
                for (int s = 0; s < 32; ++s) {
                    const uint32_t b = __ballot_sync(0xFFFFFFFFu, (code[s] >> bit) & 1u);
                    if (lane == s) mine = b;
                }
                if (word < words) out[(int64_t)j * words + word] = mine;
            }
        }
        __syncwarp();  // everyone is done with this slot before the copy after next lands in it
    }
    cp_async_wait<0>();
}

// ---- server average of bit-plane messages: thread = one word (32 entries), staged through shared memory
__global__ void __launch_bounds__(kBitThreads)
aggregate_bitwise_kernel(const uint32_t* __restrict__ planes, const float* __restrict__ gmax,
                         const int32_t* __restrict__ level, const double* __restrict__ p_sel, BitSchedule sc,
                         int w_max, int64_t words, int M, int64_t d, float* __restrict__ out) {
    __shared__ float sh_out[kBitThreads / 32][32][33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float inv_M = 1.0f / (float)M;
    const int64_t nblk = (words + kBitThreads - 1) / kBitThreads;
    for (int64_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
        const int64_t word = blk * kBitThreads + threadIdx.x;
        float acc[32];
#pragma unroll
        for (int t = 0; t < 32; ++t) acc[t] = 0.0f;
        // the sign word and the first magnitude plane of the next worker are loaded before this worker's are used
        uint32_t sgn_n = 0, pw1_n = 0;
        auto preload = [&](int mm) {
            if (mm < M && level[mm] >= 0 && word < words) {
                const uint32_t* pm = planes + (int64_t)mm * (1 + w_max) * words;
                sgn_n = pm[word];
                pw1_n = pm[words + word];
            } else {
                sgn_n = 0;
                pw1_n = 0;
            }
        };
        preload(0);
        for (int m = 0; m < M; ++m) {  // fixed worker order
            const int lv = level[m];
            const uint32_t sgn = sgn_n, pw1 = pw1_n;
            preload(m + 1);
            if (lv < 0) continue;
            const int w = sc.width[lv];
            // value of one unit of the field: 2^{-b_l} gmax / p_l
            const float unit = (float)(ldexp((double)gmax[m], -sc.bits[lv]) / p_sel[m]);
            // A word whose fields are all zero adds +-0 to every entry, which changes nothing: it is skipped.  The
            // high levels of a heavy-tailed gradient are almost all zero, so whole warps skip.
            if (w == 1) {  // the paper's case: one information bit and one sign bit per entry
                if (pw1 != 0u) {
                    const uint32_t ub = __float_as_uint(unit);
#pragma unroll
                    for (int t = 0; t < 32; ++t) {
                        const uint32_t on = 0u - ((pw1 >> t) & 1u);
                        acc[t] += __uint_as_float((ub & on) ^ (((sgn >> t) & 1u) << 31));
                    }
                }
            } else if (w <= 8) {
                // fields of at most 8 bits: each plane word is spread into the 32 field bytes, four bits per
                // multiply ((nibble * 0x00204081) & 0x01010101 puts bit i of the nibble at bit 0 of byte i)
                const uint32_t* pm = planes + (int64_t)m * (1 + w_max) * words;
                uint32_t pw[8], any = pw1;
                pw[0] = pw1;
#pragma unroll
                for (int j = 2; j <= 8; ++j) {
                    pw[j - 1] = (j <= w && word < words) ? pm[(int64_t)j * words + word] : 0u;
                    any |= pw[j - 1];
                }
                if (any != 0u) {
                    uint32_t fb[8] = {};
#pragma unroll
                    for (int j = 1; j <= 8; ++j) {
                        if (j <= w) {
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                fb[c] |= ((((pw[j - 1] >> (4 * c)) & 0xFu) * 0x00204081u) & 0x01010101u) << (w - j);
                        }
                    }
#pragma unroll
                    for (int t = 0; t < 32; ++t) {
                        const uint32_t f = (fb[t >> 2] >> (8 * (t & 3))) & 0xFFu;
                        const float ff = __uint_as_float(0x4B000000u | f) - 8388608.0f;  // exact integer-to-float through 2^23
                        acc[t] += __uint_as_float(__float_as_uint(ff * unit) ^ (((sgn >> t) & 1u) << 31));
                    }
                }
            } else {
                const uint32_t* pm = planes + (int64_t)m * (1 + w_max) * words;
                uint32_t f[32];
#pragma unroll
                for (int t = 0; t < 32; ++t) f[t] = (pw1 >> t) & 1u;
                for (int j = 2; j <= w; ++j) {
                    const uint32_t pw = (word < words) ? pm[(int64_t)j * words + word] : 0u;
#pragma unroll
                    for (int t = 0; t < 32; ++t) f[t] = (f[t] << 1) | ((pw >> t) & 1u);
                }
#pragma unroll
                for (int t = 0; t < 32; ++t) {
                    // f < 2^23: exact integer-to-float through the 2^23 offset, without the conversion unit
                    const float ff = __uint_as_float(0x4B000000u | f[t]) - 8388608.0f;
                    acc[t] += __uint_as_float(__float_as_uint(ff * unit) ^ (((sgn >> t) & 1u) << 31));
                }
            }
        }
        // transpose through shared memory so that the 32 floats of a word leave as one 128-byte row
#pragma unroll
        for (int t = 0; t < 32; ++t) sh_out[warp][lane][t] = acc[t] * inv_M;
        __syncwarp();
        const int64_t wbase = blk * kBitThreads + warp * 32;
#pragma unroll 4
        for (int r = 0; r < 32; ++r) {
            const int64_t i = (wbase + r) * 32 + lane;
            if (i < d) out[i] = sh_out[warp][r][lane];
        }
        __syncwarp();
    }
}

BitSchedule make_schedule(const int32_t* b, int L) {
    BitSchedule sc = {};
    sc.L = L;
    sc.B = b[L - 1];
    for (int l = 0; l < L; ++l) {
        const int w = b[l] - (l ? b[l - 1] : 0);
        sc.bits[l] = b[l];
        sc.width[l] = w;
        sc.shift[l] = sc.B - b[l];
        sc.mask[l] = (w >= 32) ? 0xFFFFFFFFu : ((1u << w) - 1u);
    }
    return sc;
}

int bit_blocks(const Workspace& ws, int64_t d, int vec, int M, int waves) {
    const int64_t nvec = (d + vec - 1) / vec;
    const int64_t by_work = (nvec + (int64_t)kSweepThreads * 4 - 1) / ((int64_t)kSweepThreads * 4);
    int64_t by_sm = ((int64_t)ws.sm_count * waves) / M;  // rounded down: one block too many per worker costs a whole extra wave
    int64_t nb = by_work < by_sm ? by_work : by_sm;
    return (int)(nb < 1 ? 1 : nb);
}

}  // namespace

int configure_bit_kernels() {
    const int smem = (kBitThreads / 32) * (2 * 1024 * 4 + 1024);
    if (cudaFuncSetAttribute(bit_pack_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
        cudaFuncSetAttribute(bit_pack_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return MLMC_OK;
}

void launch_absmax(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, cudaStream_t s) {
    cudaMemsetAsync(ws.gmax_bits, 0, (size_t)M * sizeof(uint32_t), s);
    LaunchScope t(ws, K_ABSMAX, s);
    if (dtype == MLMC_BF16) {
        const int nb = bit_blocks(ws, d, 8, M, 8);
        absmax_kernel<bf16_t><<<dim3(nb, M), kSweepThreads, 0, s>>>(static_cast<const bf16_t*>(g), d, ld, ws.gmax_bits,
                                                                    ws.status, ws.worker_err);
    } else {
        const int nb = bit_blocks(ws, d, 4, M, 8);
        absmax_kernel<float><<<dim3(nb, M), kSweepThreads, 0, s>>>(static_cast<const float*>(g), d, ld, ws.gmax_bits,
                                                                   ws.status, ws.worker_err);
    }
}

template <typename T, typename Acc>
static void launch_bit_stats_t(Workspace& ws, const T* g, int64_t d, int M, int64_t ld, const BitSchedule& sc, int nb,
                               cudaStream_t s) {
    dim3 grid(nb, M);
#define MLMC_BIT_STATS(LM)                                                                                          \
    bit_stats_kernel<T, LM, Acc><<<grid, kSweepThreads, 0, s>>>(g, d, ld, ws.gmax_bits, sc, ws.S_partial, ws.stat_ctas, \
                                                               ws.worker_err)
    if (sc.L <= 4) MLMC_BIT_STATS(4);
    else if (sc.L <= 6) MLMC_BIT_STATS(6);
    else if (sc.L <= 8) MLMC_BIT_STATS(8);
    else if (sc.L <= 16) MLMC_BIT_STATS(16);
    else MLMC_BIT_STATS(23);
#undef MLMC_BIT_STATS
}

void launch_bit_stats(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* b, int L,
                      cudaStream_t s) {
    const BitSchedule sc = make_schedule(b, L);
    cudaMemsetAsync(ws.S_partial, 0, (size_t)M * ws.stat_ctas * kMaxLevels * sizeof(unsigned long long), s);
    int nb = bit_blocks(ws, d, dtype == MLMC_BF16 ? 8 : 4, M, 4);
    if (nb > ws.stat_ctas) nb = ws.stat_ctas;
    ws.cur_stat_ctas = nb;
    // 32-bit sums are exact while f^2 < 2^16 and a thread adds fewer than 2^16 of them
    const int vec = dtype == MLMC_BF16 ? 8 : 4;
    const int64_t vec_per_block = ((d + vec - 1) / vec + nb - 1) / nb;
    const int64_t per_thread = ((vec_per_block + kSweepThreads - 1) / kSweepThreads + 1) * vec;
    int w_top = 0;
    for (int l = 0; l < L; ++l) w_top = sc.width[l] > w_top ? sc.width[l] : w_top;
    const bool narrow = w_top <= 8 && per_thread < 65536;
    LaunchScope t(ws, K_BIT_STATS, s);
    if (dtype == MLMC_BF16) {
        if (narrow) launch_bit_stats_t<bf16_t, uint32_t>(ws, static_cast<const bf16_t*>(g), d, M, ld, sc, nb, s);
        else launch_bit_stats_t<bf16_t, unsigned long long>(ws, static_cast<const bf16_t*>(g), d, M, ld, sc, nb, s);
    } else {
        if (narrow) launch_bit_stats_t<float, uint32_t>(ws, static_cast<const float*>(g), d, M, ld, sc, nb, s);
        else launch_bit_stats_t<float, unsigned long long>(ws, static_cast<const float*>(g), d, M, ld, sc, nb, s);
    }
}

void launch_bit_probs_draw(Workspace& ws, int M, const int32_t* b, int L, bool adaptive, bool need_delta,
                           uint64_t seed, uint64_t step, const mlmc_bit_msgs* out, cudaStream_t s) {
    const BitSchedule sc = make_schedule(b, L);
    LaunchScope t(ws, K_BIT_DRAW, s);
    bit_probs_draw_kernel<<<M, 32, 0, s>>>(
        sc, ws.gmax_bits, ws.S_partial, ws.cur_stat_ctas, ws.stat_ctas, ws.p_fixed, adaptive ? 1 : 0, need_delta ? 1 : 0,
        seed, step, M, ws.p_all, ws.delta_all, ws.u_dev, ws.bit_level, out ? out->gmax : nullptr,
        out ? out->level : nullptr, out ? out->p_sel : nullptr, out ? out->w_max : 0, out ? 1 : 0, ws.status,
        ws.worker_err);
}

template <typename T>
static void launch_bit_pack_t(Workspace& ws, const T* g, int64_t d, int M, int64_t ld, const BitSchedule& sc,
                              const mlmc_bit_msgs& out, cudaStream_t s) {
    const int64_t words = (d + 31) / 32;
    const int64_t ngroups = (words + 31) / 32;
    const int64_t by_work = (ngroups + (kBitThreads / 32) - 1) / (kBitThreads / 32);
    const size_t smem = (kBitThreads / 32) * (2 * 1024 * sizeof(T) + 1024);
    int w_top = 0, w_low = 64;
    for (int l = 0; l < sc.L; ++l) {
        w_top = sc.width[l] > w_top ? sc.width[l] : w_top;
        w_low = sc.width[l] < w_low ? sc.width[l] : w_low;
    }
    if (w_low <= 8) {  // some level has a field of at most 8 bits
        int64_t nb = ((int64_t)ws.sm_count * 3) / M;  // persistent: three resident blocks per SM, rounded down
        if (nb > by_work) nb = by_work;
        if (nb < 1) nb = 1;
        LaunchScope t(ws, K_BIT_PACK, s);
        bit_pack_kernel<T, false><<<dim3((unsigned)nb, M), kBitThreads, smem, s>>>(g, d, ld, ws.gmax_bits, sc, ws.bit_level,
                                                                                out.planes, out.w_max, words);
    }
    if (w_top > 8) {  // some level has a wider field
        int64_t nb = ((int64_t)ws.sm_count * 2) / M;  // two resident blocks per SM, rounded down
        if (nb > by_work) nb = by_work;
        if (nb < 1) nb = 1;
        LaunchScope t(ws, K_BIT_PACK_WIDE, s);
        bit_pack_kernel<T, true><<<dim3((unsigned)nb, M), kBitThreads, smem, s>>>(g, d, ld, ws.gmax_bits, sc, ws.bit_level,
                                                                               out.planes, out.w_max, words);
    }
}

void launch_bit_pack(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* b, int L,
                     const mlmc_bit_msgs& out, cudaStream_t s) {
    const BitSchedule sc = make_schedule(b, L);
    if (dtype == MLMC_BF16)
        launch_bit_pack_t<bf16_t>(ws, static_cast<const bf16_t*>(g), d, M, ld, sc, out, s);
    else
        launch_bit_pack_t<float>(ws, static_cast<const float*>(g), d, M, ld, sc, out, s);
}

void launch_aggregate_bitwise(Workspace& ws, const mlmc_bit_msgs& msgs, const int32_t* b, int L, int M, int64_t d,
                              float* out, cudaStream_t s) {
    const BitSchedule sc = make_schedule(b, L);
    const int64_t words = (d + 31) / 32;
    int64_t nb = (words + kBitThreads - 1) / kBitThreads;
    // whole waves only: every block does the same number of iterations, so a partial last wave costs a full one
    int resident = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, aggregate_bitwise_kernel, kBitThreads, 0) != cudaSuccess ||
        resident < 1)
        resident = 1;
    const int64_t cap = (int64_t)ws.sm_count * resident * 2;
    if (nb > cap) nb = cap;
    LaunchScope t(ws, K_AGG_BIT, s);
    aggregate_bitwise_kernel<<<(unsigned)nb, kBitThreads, 0, s>>>(msgs.planes, msgs.gmax, msgs.level, msgs.p_sel, sc,
                                                                  msgs.w_max, words, M, d, out);
}

}  // namespace mlmc
