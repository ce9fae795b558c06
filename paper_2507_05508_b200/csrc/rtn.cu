// MLMC with round-to-nearest levels (Sec. 3.2 end, App. G).
//
//   C^l(v) = clip(delta^l round(v / delta^l), -c, c),  delta^l = 2c / (2^{r_l} - 1),  c = max_i |v_i|;
// the top level is the identity (Def. 3.1) and C^{-1} = 0.  The residual C^l - C^{l-1} is dense and has no band or
// bit-plane structure, so the adaptive probabilities (Lemma 3.4, Alg. 3) need ||C^l - C^{l-1}|| of every level from
// one sweep: every thread keeps one fp64 accumulator per level in registers (every entry contributes to every
// level, so no accumulator has to be selected).  Then the draw, and a sweep that writes the dense message.
//
// The rounding decides an integer, so its arithmetic is fixed (the same on the host checker): with
// inv = fl32((2^r - 1) / (2c)) and delta = fl32(2c / (2^r - 1)), t = fl32(v inv), k = t rounded to nearest, ties to
// even, C = clip(fl32(k delta), -c, c).  Residuals, norms and the scaling by 1/p are fp64.
#include "common.cuh"

namespace mlmc {

namespace {

constexpr int kRtnThreads = 256;
constexpr int kRtnMaxLevels = 17;  // widths 1..16 strictly increasing, plus the identity

struct RtnSchedule {
    int L;                  // levels, the last one is the identity
    int r[kRtnMaxLevels];   // widths of levels 0..L-2
};

struct RtnGrid {
    float inv, delta;
};

__device__ __forceinline__ RtnGrid rtn_grid(float c, int r) {
    const double steps = (double)((1u << r) - 1u);
    RtnGrid gq;
    gq.inv = (float)(steps / (2.0 * (double)c));
    gq.delta = (float)(2.0 * (double)c / steps);
    return gq;
}

__device__ __forceinline__ float rtn_value(float v, float c, RtnGrid gq) {
    const float t = __fmul_rn(v, gq.inv);
    // to nearest, ties to even: |t| <= 2^15 (r <= 16), so adding and subtracting 1.5 * 2^23 rounds t to an integer in
    // the adder, with the default rounding mode, without the conversion unit
    const float k = __fadd_rn(__fadd_rn(t, 12582912.0f), -12582912.0f);
    return fminf(fmaxf(__fmul_rn(k, gq.delta), -c), c);
}

// Residual energies of every level: partial[m][block][l] = sum over the block's entries of (C^l - C^{l-1})^2.
template <typename T, int LMAX>
__global__ void __launch_bounds__(kRtnThreads)
rtn_stats_kernel(const T* __restrict__ g, int64_t d, int64_t ld, const uint32_t* __restrict__ gmax_bits, RtnSchedule sc,
                 double* __restrict__ partial, int rtn_ctas, const int* worker_err) {
    using Tr = ElemTraits<T>;
    __shared__ double sh_red[kRtnThreads / 32];
    const int m = blockIdx.y;
    if (worker_err[m]) return;
    const float c = __uint_as_float(gmax_bits[m]);
    double acc[LMAX];
    RtnGrid grid[LMAX];
#pragma unroll
    for (int l = 0; l < LMAX; ++l) {
        acc[l] = 0.0;
        grid[l] = rtn_grid(c > 0.0f ? c : 1.0f, (l < sc.L - 1) ? sc.r[l] : 1);
    }
    if (c > 0.0f) {
        const T* row = g + (int64_t)m * ld;
        int64_t v0, v1;
        block_vector_range(d, Tr::kVec, blockIdx.x, gridDim.x, &v0, &v1);
        auto take = [&](uint32_t bits) {
            const float v = Tr::value(bits);
            double prev = 0.0;  // C^{l-1}
#pragma unroll
            for (int l = 0; l < LMAX; ++l) {
                // levels past the identity repeat it: their residual is v - v = 0
                const double cur = (l < sc.L - 1) ? (double)rtn_value(v, c, grid[l]) : (double)v;
                const double res = cur - prev;
                acc[l] = fma(res, res, acc[l]);
                prev = cur;
            }
        };
        constexpr int kBatch = 2;
        const int64_t full_end = min(v1, d / Tr::kVec);
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
    // fixed-order reduction: shuffle tree per warp, then the warp sums in warp order
#pragma unroll
    for (int l = 0; l < LMAX; ++l) {
        if (l >= sc.L) break;
        double x = acc[l];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
        if ((threadIdx.x & 31) == 0) sh_red[threadIdx.x >> 5] = x;
        __syncthreads();
        if (threadIdx.x == 0) {
            double s = 0.0;
            for (int w = 0; w < kRtnThreads / 32; ++w) s += sh_red[w];
            partial[((int64_t)m * rtn_ctas + blockIdx.x) * kMaxLevels + l] = s;
        }
        __syncthreads();
    }
}

// Delta_l, p_l = Delta_l / sum Delta (Lemma 3.4) or the given p, the draw, the message header.
__global__ void rtn_probs_draw_kernel(int L, const uint32_t* gmax_bits, const double* partial, int n_partials,
                                      int rtn_ctas, const double* p_fixed, int adaptive, int have_stats, uint64_t seed,
                                      uint64_t step, int M, double* p_all, double* delta_all, double* u_dev,
                                      int32_t* bit_level, float* out_c, int32_t* out_level, double* out_p_sel,
                                      const int* worker_err) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    if (worker_err[m]) {
        bit_level[m] = -1;
        if (out_level) {
            out_level[m] = -1;
            out_p_sel[m] = 0.0;
            out_c[m] = 0.0f;
        }
        return;
    }
    double p[kRtnMaxLevels], s = 0.0;
    for (int l = 0; l < L; ++l) {
        double e = 0.0;
        if (have_stats)
            for (int c = 0; c < n_partials; ++c) e += partial[((int64_t)m * rtn_ctas + c) * kMaxLevels + l];  // block order
        const double dl = sqrt(e);
        delta_all[m * kMaxLevels + l] = dl;
        p[l] = dl;
        s += dl;
    }
    for (int l = 0; l < L; ++l) {
        p[l] = adaptive ? ((s > 0.0) ? p[l] / s : (l == 0 ? 1.0 : 0.0)) : p_fixed[l];
        p_all[m * kMaxLevels + l] = p[l];
    }
    const double u = counter_uniform(seed, step, (uint64_t)m);
    u_dev[m] = u;
    const int level = draw_from_probs(p, L, u);
    bit_level[m] = level;
    if (out_level) {
        out_level[m] = level;
        out_p_sel[m] = p[level];
        out_c[m] = __uint_as_float(gmax_bits[m]);
    }
}

// The dense message of the drawn level: val_i = (C^l - C^{l-1})_i / p_l, rounded to fp32 once.
template <typename T>
__global__ void __launch_bounds__(kRtnThreads)
rtn_emit_kernel(const T* __restrict__ g, int64_t d, int64_t ld, const uint32_t* __restrict__ gmax_bits, RtnSchedule sc,
                const int32_t* __restrict__ bit_level, const double* __restrict__ p_all, float* __restrict__ val,
                int64_t ldv) {
    using Tr = ElemTraits<T>;
    const int m = blockIdx.y;
    const int level = bit_level[m];
    if (level < 0) return;
    const float c = __uint_as_float(gmax_bits[m]);
    const double p = p_all[m * kMaxLevels + level];
    const double inv_p = p > 0.0 ? 1.0 / p : 0.0;
    const bool top = level == sc.L - 1, first = level == 0;
    const RtnGrid g_hi = rtn_grid(c > 0.0f ? c : 1.0f, top ? 1 : sc.r[level]);
    const RtnGrid g_lo = rtn_grid(c > 0.0f ? c : 1.0f, first ? 1 : sc.r[level - 1]);
    const T* row = g + (int64_t)m * ld;
    float* out = val + (int64_t)m * ldv;
    auto residual = [&](uint32_t bits) -> float {
        const float v = Tr::value(bits);
        if (!(c > 0.0f)) return 0.0f;
        const double hi = top ? (double)v : (double)rtn_value(v, c, g_hi);
        const double lo = first ? 0.0 : (double)rtn_value(v, c, g_lo);
        return (float)((hi - lo) * inv_p);
    };
    const int64_t nvec = (d + Tr::kVec - 1) / Tr::kVec;
    const bool vec_ok = (ldv % 4 == 0);
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += (int64_t)gridDim.x * blockDim.x) {
        const int64_t base = v * Tr::kVec;
        if (base + Tr::kVec <= d && vec_ok) {
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(row) + v);
            if constexpr (Tr::kVec == 4) {
                reinterpret_cast<float4*>(out + base)[0] = make_float4(residual(q.x), residual(q.y), residual(q.z), residual(q.w));
            } else {
                reinterpret_cast<float4*>(out + base)[0] =
                    make_float4(residual(q.x & 0xFFFFu), residual(q.x >> 16), residual(q.y & 0xFFFFu), residual(q.y >> 16));
                reinterpret_cast<float4*>(out + base)[1] =
                    make_float4(residual(q.z & 0xFFFFu), residual(q.z >> 16), residual(q.w & 0xFFFFu), residual(q.w >> 16));
            }
        } else {
            for_each_in_vector<T>(row, v, d, [&](int64_t i, uint32_t bits) { out[i] = residual(bits); });
        }
    }
}

// Server average of dense messages: out[i] = (1/M) sum_m val[m][i] in worker order.
__global__ void __launch_bounds__(kRtnThreads)
aggregate_dense_kernel(const float* __restrict__ val, const int32_t* __restrict__ level, int M, int64_t d, int64_t ldv,
                       float* __restrict__ out) {
    const float inv_M = 1.0f / (float)M;
    const bool vec_ok = (ldv % 4 == 0) && (d % 4 == 0);
    if (vec_ok) {
        const int64_t n4 = d / 4;
        for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += (int64_t)gridDim.x * blockDim.x) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int m = 0; m < M; ++m) {
                if (level[m] < 0) continue;
                const float4 x = __ldg(reinterpret_cast<const float4*>(val + (int64_t)m * ldv) + v);
                a.x += x.x; a.y += x.y; a.z += x.z; a.w += x.w;
            }
            a.x *= inv_M; a.y *= inv_M; a.z *= inv_M; a.w *= inv_M;
            reinterpret_cast<float4*>(out)[v] = a;
        }
    } else {
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += (int64_t)gridDim.x * blockDim.x) {
            float a = 0.f;
            for (int m = 0; m < M; ++m)
                if (level[m] >= 0) a += val[(int64_t)m * ldv + i];
            out[i] = a * inv_M;
        }
    }
}

RtnSchedule make_rtn_schedule(const int32_t* r, int L) {
    RtnSchedule sc = {};
    sc.L = L;
    for (int l = 0; l + 1 < L; ++l) sc.r[l] = r[l];
    return sc;
}

int rtn_blocks(const Workspace& ws, int64_t d, int vec, int M, int per_sm) {
    const int64_t nvec = (d + vec - 1) / vec;
    const int64_t by_work = (nvec + (int64_t)kRtnThreads * 4 - 1) / ((int64_t)kRtnThreads * 4);
    int64_t by_sm = ((int64_t)ws.sm_count * per_sm) / M;
    int64_t nb = by_work < by_sm ? by_work : by_sm;
    return (int)(nb < 1 ? 1 : nb);
}

}  // namespace

void launch_rtn_stats(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* r, int L,
                      cudaStream_t s) {
    const RtnSchedule sc = make_rtn_schedule(r, L);
    int nb = rtn_blocks(ws, d, dtype == MLMC_BF16 ? 8 : 4, M, 8);
    if (nb > ws.rtn_ctas) nb = ws.rtn_ctas;
    ws.cur_rtn_ctas = nb;
    dim3 grid(nb, M);
    LaunchScope t(ws, K_RTN_STATS, s);
#define MLMC_RTN_STATS(TT, LM)                                                                                      \
    rtn_stats_kernel<TT, LM><<<grid, kRtnThreads, 0, s>>>(static_cast<const TT*>(g), d, ld, ws.gmax_bits, sc,       \
                                                         ws.rtn_partial, ws.rtn_ctas, ws.worker_err)
    if (dtype == MLMC_BF16) {
        if (L <= 6) MLMC_RTN_STATS(bf16_t, 6);
        else MLMC_RTN_STATS(bf16_t, kRtnMaxLevels);
    } else {
        if (L <= 6) MLMC_RTN_STATS(float, 6);
        else MLMC_RTN_STATS(float, kRtnMaxLevels);
    }
#undef MLMC_RTN_STATS
}

void launch_rtn_probs_draw(Workspace& ws, int M, int L, bool adaptive, bool have_stats, uint64_t seed, uint64_t step,
                           const mlmc_rtn_msgs* out, cudaStream_t s) {
    LaunchScope t(ws, K_RTN_DRAW, s);
    rtn_probs_draw_kernel<<<(M + 63) / 64, 64, 0, s>>>(L, ws.gmax_bits, ws.rtn_partial, ws.cur_rtn_ctas, ws.rtn_ctas,
                                                      ws.p_fixed, adaptive ? 1 : 0, have_stats ? 1 : 0, seed, step, M,
                                                      ws.p_all, ws.delta_all, ws.u_dev, ws.bit_level,
                                                      out ? out->c : nullptr, out ? out->level : nullptr,
                                                      out ? out->p_sel : nullptr, ws.worker_err);
}

void launch_rtn_emit(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* r, int L,
                     const mlmc_rtn_msgs& out, cudaStream_t s) {
    const RtnSchedule sc = make_rtn_schedule(r, L);
    const int nb = rtn_blocks(ws, d, dtype == MLMC_BF16 ? 8 : 4, M, 16);
    dim3 grid(nb, M);
    LaunchScope t(ws, K_RTN_EMIT, s);
    if (dtype == MLMC_BF16)
        rtn_emit_kernel<bf16_t><<<grid, kRtnThreads, 0, s>>>(static_cast<const bf16_t*>(g), d, ld, ws.gmax_bits, sc,
                                                            ws.bit_level, ws.p_all, out.val, out.ldv);
    else
        rtn_emit_kernel<float><<<grid, kRtnThreads, 0, s>>>(static_cast<const float*>(g), d, ld, ws.gmax_bits, sc,
                                                           ws.bit_level, ws.p_all, out.val, out.ldv);
}

void launch_aggregate_dense(Workspace& ws, const float* val, const int32_t* level, int M, int64_t d, int64_t ldv,
                            float* out, cudaStream_t s) {
    int64_t nb = (d / 4 + kRtnThreads - 1) / kRtnThreads;
    const int64_t cap = (int64_t)ws.sm_count * 16;
    if (nb > cap) nb = cap;
    if (nb < 1) nb = 1;
    LaunchScope t(ws, K_AGG_DENSE, s);
    aggregate_dense_kernel<<<(unsigned)nb, kRtnThreads, 0, s>>>(val, level, M, d, ldv, out);
}

}  // namespace mlmc
