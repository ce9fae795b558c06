// MLMC gradient-compression oracle: TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded CPU statement of what the GPU library computes, written from
// the paper's definitions.  It shares no code with the CUDA path and must never be called from
// the product path; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
//
// Notation (paper level l = 1..L with g^0 = 0  <->  here level l = 0..L-1 with k_{-1} = 0, b_{-1} = 0):
//   Top-k compressor C^l keeps the k_l entries of largest |g| (Sec. 2.2 "Top-k"); the order is
//   total: |g| descending as real numbers, equal magnitudes by ascending index.
//   band_l = coordinates of rank (k_{l-1}, k_l]  = support of C^l(g) - C^{l-1}(g) (Sec. 3, remark
//   after Alg. 2; Sec. 3.2).
//   MLMC estimate  g~ = g^0 + (1/p^l)(g^l - g^{l-1}),  g^0 = 0,  l ~ p        (Eq. 5, Alg. 2/3)
//   adaptive p^l = Delta^l / sum_l' Delta^l',  Delta^l = ||g^l - g^{l-1}||_2  (Lemma 3.4)
//   fixed-point compressor: entries divided by the largest magnitude, written as sign + B
//   fractional bits, level l keeps the b_l most significant bits (Sec. 3.1, Eq. 6).
//   floating-point compressor: sign and exponent are kept, level l keeps the m_l most significant
//   mantissa bits (Sec. 2.2 "Floating-point compressors", App. B).
//   s-Top-k: Top-(s k) of the sorted vector, i.e. the uniform schedule k_l = s (l + 1) (Sec. 2.2, App. D).
//   RTN: C^l(v) = clip(delta^l round(v / delta^l), -c, c), delta^l = 2c / (2^l - 1) (Sec. 3.2, App. G).
//   server: (1/M) sum_i g~_i                                                  (Alg. 2, "Server aggregates")
//
// Every function here is pinned by tests/test_oracle_*.py against closed forms, brute force on
// tiny inputs and the identities of Lemma 3.2 / 3.3 / 3.4; nothing is "parity unpinned".
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC  (no fast-math: IEEE float division matters).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {

constexpr int DT_F32 = 0;
constexpr int DT_BF16 = 1;

constexpr int ORA_OK = 0;
constexpr int ORA_ERR_ARG = -1;
constexpr int ORA_ERR_SCHEDULE = -2;
constexpr int ORA_ERR_PROB = -3;
constexpr int ORA_ERR_CAPACITY = -4;
constexpr int ORA_ERR_NONFINITE = -5;

// bf16 -> fp32 is exact: bf16 is the upper half of the fp32 encoding.
inline float widen_bf16(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

inline float elem(const void* g, int dtype, int64_t i) {
    if (dtype == DT_BF16) return widen_bf16(static_cast<const uint16_t*>(g)[i]);
    return static_cast<const float*>(g)[i];
}

inline bool sign_bit(float x) {
    uint32_t u;
    std::memcpy(&u, &x, sizeof u);
    return (u >> 31) != 0;
}

// ---- counter-based uniform: three chained SplitMix64 output rounds over (seed, step, worker) ----
constexpr uint64_t GOLDEN = 0x9E3779B97F4A7C15ull;

inline uint64_t splitmix_finalize(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

inline uint64_t counter_hash(uint64_t seed, uint64_t step, uint64_t worker) {
    uint64_t h = splitmix_finalize(seed + GOLDEN);
    h = splitmix_finalize(h + step + GOLDEN);
    h = splitmix_finalize(h + worker + GOLDEN);
    return h;
}

inline double uniform01(uint64_t seed, uint64_t step, uint64_t worker) {
    return static_cast<double>(counter_hash(seed, step, worker) >> 11) * 0x1.0p-53;
}

// ---- inverse-CDF level draw ("Sample l ~ p^l", Alg. 2 / Alg. 3) ----
// cdf_j = p_0 + ... + p_j accumulated in ascending j; the cdf of the last level with p > 0 (and of
// every level after it) is 1 exactly; l* = min{ j : u < cdf_j }.  margin = distance from u to the
// nearest interior cdf boundary (boundaries equal to 1 cannot be crossed because u < 1).
void draw_level(const double* p, int L, double u, int* level, double* margin) {
    int j_last = -1;
    for (int j = 0; j < L; ++j)
        if (p[j] > 0.0) j_last = j;
    double c = 0.0, mg = std::numeric_limits<double>::infinity();
    int lv = -1;
    for (int j = 0; j < L; ++j) {
        c += p[j];
        const bool forced = (j >= j_last);
        const double cdf = forced ? 1.0 : c;
        if (!forced) mg = std::min(mg, std::fabs(u - cdf));
        if (lv < 0 && u < cdf) lv = j;
    }
    if (lv < 0) lv = 0;  // only when every p is 0 (callers never pass that)
    *level = lv;
    *margin = mg;
}

int check_finite(const void* g, int dtype, int64_t d) {
    for (int64_t i = 0; i < d; ++i)
        if (!std::isfinite(elem(g, dtype, i))) return ORA_ERR_NONFINITE;
    return ORA_OK;
}

int check_topk_schedule(const int64_t* k, int L, int64_t d) {
    if (L < 1) return ORA_ERR_ARG;
    int64_t prev = 0;
    for (int l = 0; l < L; ++l) {
        if (k[l] < prev || k[l] > d) return ORA_ERR_SCHEDULE;
        prev = k[l];
    }
    // Def. 3.1: the highest level is the identity, i.e. Top-k with k = d.
    return k[L - 1] == d ? ORA_OK : ORA_ERR_SCHEDULE;
}

int check_bit_schedule(const int32_t* b, int L) {
    if (L < 1) return ORA_ERR_ARG;
    int prev = 0;
    for (int l = 0; l < L; ++l) {
        if (b[l] <= prev || b[l] > 23) return ORA_ERR_SCHEDULE;
        prev = b[l];
    }
    return ORA_OK;
}

// fixed p: every entry must be > 0 (Lemma 3.2 asks for non-zero probabilities); normalised in fp64.
int normalise_fixed(const double* p_in, int L, double* p) {
    double s = 0.0;
    for (int l = 0; l < L; ++l) {
        if (!(p_in[l] > 0.0) || !std::isfinite(p_in[l])) return ORA_ERR_PROB;
        s += p_in[l];
    }
    if (std::fabs(s - 1.0) > 1e-9) return ORA_ERR_PROB;
    for (int l = 0; l < L; ++l) p[l] = p_in[l] / s;
    return ORA_OK;
}

// adaptive p (Lemma 3.4).  An all-zero residual family (sum Delta = 0) puts everything on level 0.
void adaptive_probs(const double* delta, int L, double* p) {
    double s = 0.0;
    for (int l = 0; l < L; ++l) s += delta[l];
    if (!(s > 0.0)) {
        for (int l = 0; l < L; ++l) p[l] = (l == 0) ? 1.0 : 0.0;
        return;
    }
    for (int l = 0; l < L; ++l) p[l] = delta[l] / s;
}

// Full stable sort of the coordinates by |g| descending; stable => equal magnitudes keep ascending index.
void rank_by_magnitude(const void* g, int dtype, int64_t d, std::vector<uint32_t>& perm) {
    perm.resize(static_cast<size_t>(d));
    std::iota(perm.begin(), perm.end(), 0u);
    std::vector<float> mag(static_cast<size_t>(d));
    for (int64_t i = 0; i < d; ++i) mag[static_cast<size_t>(i)] = std::fabs(elem(g, dtype, i));
    std::stable_sort(perm.begin(), perm.end(),
                     [&mag](uint32_t a, uint32_t b) { return mag[a] > mag[b]; });
}

}  // namespace

extern "C" {

uint64_t mlmc_oracle_hash(uint64_t seed, uint64_t step, uint64_t worker) {
    return counter_hash(seed, step, worker);
}

double mlmc_oracle_uniform(uint64_t seed, uint64_t step, uint64_t worker) {
    return uniform01(seed, step, worker);
}

int mlmc_oracle_draw(const double* p, int L, double u, int* level, double* margin) {
    if (L < 1) return ORA_ERR_ARG;
    draw_level(p, L, u, level, margin);
    return ORA_OK;
}

// perm[r] = coordinate of rank r+1 in the total order.
int mlmc_oracle_rank(const void* g, int dtype, int64_t d, uint32_t* perm) {
    if (d < 0 || d > 0xFFFFFFFFll) return ORA_ERR_ARG;
    if (int rc = check_finite(g, dtype, d)) return rc;
    std::vector<uint32_t> pv;
    rank_by_magnitude(g, dtype, d, pv);
    std::copy(pv.begin(), pv.end(), perm);
    return ORA_OK;
}

// One worker's MLMC-Top-k message.
//   p_in == NULL  -> adaptive probabilities (Lemma 3.4);  else fixed p (host array of L).
//   force_level >= 0 replaces the draw (used to enumerate all levels in the unbiasedness pins);
//   the probabilities are still the ones the rule gives.
// Outputs (any may be NULL except level/p_sel/count): p_out[L], delta_out[L] (always the true
// band norms), u, margin, and the message (idx ascending, val = (float)((double)g_i / p_l)).
int mlmc_oracle_topk(const void* g, int dtype, int64_t d, const int64_t* k, int L, const double* p_in,
                     uint64_t seed, uint64_t step, uint64_t worker, int force_level,
                     double* p_out, double* delta_out, int32_t* level_out, double* p_sel_out,
                     double* u_out, double* margin_out,
                     int64_t* count_out, uint32_t* idx_out, float* val_out, int64_t capacity) {
    if (d < 1 || d > 0xFFFFFFFFll || !level_out || !p_sel_out || !count_out) return ORA_ERR_ARG;
    if (int rc = check_topk_schedule(k, L, d)) return rc;
    if (int rc = check_finite(g, dtype, d)) return rc;
    std::vector<double> p(static_cast<size_t>(L)), delta(static_cast<size_t>(L));
    if (p_in)
        if (int rc = normalise_fixed(p_in, L, p.data())) return rc;

    std::vector<uint32_t> perm;
    rank_by_magnitude(g, dtype, d, perm);

    // Delta_l: l2 norm of the band, summed in fp64 in ascending coordinate order.
    std::vector<uint32_t> band;
    for (int l = 0; l < L; ++l) {
        const int64_t lo = (l == 0) ? 0 : k[l - 1], hi = k[l];
        band.assign(perm.begin() + lo, perm.begin() + hi);
        std::sort(band.begin(), band.end());
        double s = 0.0;
        for (uint32_t i : band) {
            const double x = static_cast<double>(elem(g, dtype, i));
            s += x * x;
        }
        delta[static_cast<size_t>(l)] = std::sqrt(s);
    }
    if (!p_in) adaptive_probs(delta.data(), L, p.data());

    const double u = uniform01(seed, step, worker);
    int level;
    double margin;
    draw_level(p.data(), L, u, &level, &margin);
    if (force_level >= 0) {
        if (force_level >= L) return ORA_ERR_ARG;
        level = force_level;
    }
    const double p_sel = p[static_cast<size_t>(level)];

    if (p_out) std::copy(p.begin(), p.end(), p_out);
    if (delta_out) std::copy(delta.begin(), delta.end(), delta_out);
    if (u_out) *u_out = u;
    if (margin_out) *margin_out = margin;
    *level_out = level;
    *p_sel_out = p_sel;

    const int64_t lo = (level == 0) ? 0 : k[level - 1], hi = k[level];
    const int64_t n = hi - lo;
    *count_out = n;
    if (idx_out && val_out) {
        if (n > capacity) return ORA_ERR_CAPACITY;
        band.assign(perm.begin() + lo, perm.begin() + hi);
        std::sort(band.begin(), band.end());
        for (int64_t j = 0; j < n; ++j) {
            const uint32_t i = band[static_cast<size_t>(j)];
            idx_out[j] = i;
            // g^0 = 0, so the estimate is the band scaled by 1/p^l and nothing else (Eq. 5).
            val_out[j] = (p_sel > 0.0)
                             ? static_cast<float>(static_cast<double>(elem(g, dtype, i)) / p_sel)
                             : 0.0f;
        }
    }
    return ORA_OK;
}

// Fixed-point code of every entry (Sec. 3.1): e = |g| / gmax in fp32 (IEEE division),
// q = min(floor(e * 2^B), 2^B - 1).  The clamp covers |e| = 1, which B fractional bits cannot hold.
int mlmc_oracle_fixed_point_codes(const void* g, int dtype, int64_t d, int B, float* gmax_out,
                                  uint32_t* q_out) {
    if (d < 1 || B < 1 || B > 23) return ORA_ERR_ARG;
    if (int rc = check_finite(g, dtype, d)) return rc;
    float gmax = 0.0f;
    for (int64_t i = 0; i < d; ++i) gmax = std::max(gmax, std::fabs(elem(g, dtype, i)));
    *gmax_out = gmax;
    const float two_b = static_cast<float>(1u << B);
    const uint32_t qmax = (1u << B) - 1u;
    for (int64_t i = 0; i < d; ++i) {
        uint32_t q = 0;
        if (gmax > 0.0f) {
            const float e = std::fabs(elem(g, dtype, i)) / gmax;
            const float scaled = e * two_b;  // exact: power-of-two scaling, no overflow
            q = static_cast<uint32_t>(scaled);  // truncation: "discarding the least significant bits"
            if (q > qmax) q = qmax;
        }
        q_out[i] = q;
    }
    return ORA_OK;
}

// One worker's bit-wise MLMC message.  planes_out holds (1 + w_max) planes of words = ceil(d/32)
// uint32 each: plane 0 = raw sign bits, plane j (1..w_l) = bit (w_l - j) of the level's field,
// bit t of word w = coordinate 32 w + t; planes beyond 1 + w_l are left untouched.
// S_out[L] = exact sum of squared fields per level; delta_l = gmax 2^{-b_l} sqrt(S_l).
int mlmc_oracle_bitwise(const void* g, int dtype, int64_t d, const int32_t* b, int L, const double* p_in,
                        uint64_t seed, uint64_t step, uint64_t worker, int force_level,
                        double* p_out, double* delta_out, uint64_t* S_out,
                        int32_t* level_out, double* p_sel_out, double* u_out, double* margin_out,
                        float* gmax_out, uint32_t* planes_out, int32_t w_max) {
    if (d < 1 || !level_out || !p_sel_out || !gmax_out) return ORA_ERR_ARG;
    if (int rc = check_bit_schedule(b, L)) return rc;
    std::vector<double> p(static_cast<size_t>(L)), delta(static_cast<size_t>(L));
    if (p_in)
        if (int rc = normalise_fixed(p_in, L, p.data())) return rc;
    const int B = b[L - 1];
    std::vector<uint32_t> q(static_cast<size_t>(d));
    float gmax;
    if (int rc = mlmc_oracle_fixed_point_codes(g, dtype, d, B, &gmax, q.data())) return rc;

    auto field = [&](uint32_t code, int l) -> uint32_t {
        const int w = b[l] - (l ? b[l - 1] : 0);
        return (code >> (B - b[l])) & ((1u << w) - 1u);
    };
    for (int l = 0; l < L; ++l) {
        unsigned __int128 s = 0;
        for (int64_t i = 0; i < d; ++i) {
            const uint64_t f = field(q[static_cast<size_t>(i)], l);
            s += f * f;
        }
        if (S_out) S_out[l] = static_cast<uint64_t>(s);  // callers stay below 2^64 (w <= 16 or small d)
        delta[static_cast<size_t>(l)] =
            static_cast<double>(gmax) * std::ldexp(1.0, -b[l]) * std::sqrt(static_cast<double>(s));
    }
    if (!p_in) adaptive_probs(delta.data(), L, p.data());

    const double u = uniform01(seed, step, worker);
    int level;
    double margin;
    draw_level(p.data(), L, u, &level, &margin);
    if (force_level >= 0) {
        if (force_level >= L) return ORA_ERR_ARG;
        level = force_level;
    }
    if (p_out) std::copy(p.begin(), p.end(), p_out);
    if (delta_out) std::copy(delta.begin(), delta.end(), delta_out);
    if (u_out) *u_out = u;
    if (margin_out) *margin_out = margin;
    *level_out = level;
    *p_sel_out = p[static_cast<size_t>(level)];
    *gmax_out = gmax;

    if (planes_out) {
        const int w = b[level] - (level ? b[level - 1] : 0);
        if (w > w_max) return ORA_ERR_CAPACITY;
        const int64_t words = (d + 31) / 32;
        std::fill(planes_out, planes_out + (1 + w) * words, 0u);
        for (int64_t i = 0; i < d; ++i) {
            const int64_t wd = i >> 5;
            const uint32_t bit = 1u << (i & 31);
            if (sign_bit(elem(g, dtype, i))) planes_out[wd] |= bit;
            const uint32_t f = field(q[static_cast<size_t>(i)], level);
            for (int j = 1; j <= w; ++j)
                if ((f >> (w - j)) & 1u) planes_out[j * words + wd] |= bit;
        }
    }
    return ORA_OK;
}

// Decode one bit-plane message into the dense estimate (fp64): sign * f * 2^{-b_l} * gmax / p.
int mlmc_oracle_bitwise_decode(const uint32_t* planes, int64_t d, const int32_t* b, int L, int level,
                               float gmax, double p_sel, double* est_out) {
    if (level < 0 || level >= L) return ORA_ERR_ARG;
    const int w = b[level] - (level ? b[level - 1] : 0);
    const int64_t words = (d + 31) / 32;
    const double unit = std::ldexp(1.0, -b[level]) * static_cast<double>(gmax);
    for (int64_t i = 0; i < d; ++i) {
        const int64_t wd = i >> 5;
        const int t = static_cast<int>(i & 31);
        uint32_t f = 0;
        for (int j = 1; j <= w; ++j) f = (f << 1) | ((planes[j * words + wd] >> t) & 1u);
        const double mag = static_cast<double>(f) * unit;
        const double v = (p_sel > 0.0) ? mag / p_sel : 0.0;
        est_out[i] = ((planes[wd] >> t) & 1u) ? -v : v;
    }
    return ORA_OK;
}

// Server average of M Top-k messages (Alg. 2, "Server aggregates"): fp64 sums in worker order.
// scale_out (optional) = (1/M) sum_m |term|, the conditioning scale for tolerance checks.
int mlmc_oracle_aggregate_topk(int M, const int64_t* count, const uint32_t* const* idx,
                               const float* const* val, int64_t d, double* out, double* scale_out) {
    if (M < 1 || d < 1) return ORA_ERR_ARG;
    std::fill(out, out + d, 0.0);
    if (scale_out) std::fill(scale_out, scale_out + d, 0.0);
    for (int m = 0; m < M; ++m)
        for (int64_t j = 0; j < count[m]; ++j) {
            const uint32_t i = idx[m][j];
            if (static_cast<int64_t>(i) >= d) return ORA_ERR_ARG;
            out[i] += static_cast<double>(val[m][j]);
            if (scale_out) scale_out[i] += std::fabs(static_cast<double>(val[m][j]));
        }
    const double inv = 1.0 / static_cast<double>(M);
    for (int64_t i = 0; i < d; ++i) {
        out[i] *= inv;
        if (scale_out) scale_out[i] *= inv;
    }
    return ORA_OK;
}

// Server average of M bit-plane messages.
int mlmc_oracle_aggregate_bitwise(int M, const uint32_t* const* planes, const float* gmax,
                                  const int32_t* level, const double* p_sel, const int32_t* b, int L,
                                  int64_t d, double* out, double* scale_out) {
    if (M < 1 || d < 1) return ORA_ERR_ARG;
    std::fill(out, out + d, 0.0);
    if (scale_out) std::fill(scale_out, scale_out + d, 0.0);
    std::vector<double> est(static_cast<size_t>(d));
    for (int m = 0; m < M; ++m) {
        if (int rc = mlmc_oracle_bitwise_decode(planes[m], d, b, L, level[m], gmax[m], p_sel[m], est.data()))
            return rc;
        for (int64_t i = 0; i < d; ++i) {
            out[i] += est[static_cast<size_t>(i)];
            if (scale_out) scale_out[i] += std::fabs(est[static_cast<size_t>(i)]);
        }
    }
    const double inv = 1.0 / static_cast<double>(M);
    for (int64_t i = 0; i < d; ++i) {
        out[i] *= inv;
        if (scale_out) scale_out[i] *= inv;
    }
    return ORA_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Floating-point bit-wise MLMC (Sec. 2.2 "Floating-point compressors", App. B)
// ---------------------------------------------------------------------------------------------
// An entry is e = (-1)^S 2^(E - bias) (1 + sum_j m_j 2^-j); the level-l compressor truncates the
// mantissa sum to its first mb_l terms (App. B, first display).  The input here is fp32 (F = 23
// mantissa bits) or bf16 (F = 7) instead of the paper's 64-bit numbers, and the schedule
// mb_0 < ... < mb_{L-1} = F generalises the paper's unit schedule mb_l = l + 1; the top level is the
// identity (Def. 3.1).  For an entry with exponent field 0 (zero or subnormal) the leading 1 is absent
// and the scale is that of exponent field 1.
//
// Level-0 term: App. B's second moment and its lemma treat every residual as mantissa bits only,
// which holds when the always-transmitted part (sign and exponent) is the base g^0 = C^0(e) =
// (-1)^S 2^(E - bias); the estimate is g^0 + (1/p^l)(C^l - C^{l-1}) with mb_{-1} = 0.
namespace {

int float_mantissa_bits(int dtype) { return dtype == DT_BF16 ? 7 : 23; }

int check_mantissa_schedule(const int32_t* mb, int L, int F) {
    if (L < 1) return ORA_ERR_ARG;
    int prev = 0;
    for (int l = 0; l < L; ++l) {
        if (mb[l] <= prev || mb[l] > F) return ORA_ERR_SCHEDULE;
        prev = mb[l];
    }
    return mb[L - 1] == F ? ORA_OK : ORA_ERR_SCHEDULE;  // Def. 3.1: the top level is the identity
}

// C^l(e): the first `keep` mantissa digits survive, the rest are dropped (keep = 0: sign and exponent only).
double float_truncate(float x, int keep) {
    uint32_t u;
    std::memcpy(&u, &x, sizeof u);
    u &= ~((1u << (23 - keep)) - 1u);
    float y;
    std::memcpy(&y, &u, sizeof y);
    return static_cast<double>(y);
}

// App. B's lemma: p^l proportional to 2^-l for the unit schedule.  Its argument (the worst case over the mantissa
// digits) gives p^l proportional to the largest residual of the level, 2^-mb_{l-1} - 2^-mb_l, for a general one.
void float_default_probs(const int32_t* mb, int L, double* p) {
    double s = 0.0;
    for (int l = 0; l < L; ++l) {
        p[l] = std::ldexp(1.0, -(l ? mb[l - 1] : 0)) - std::ldexp(1.0, -mb[l]);
        s += p[l];
    }
    for (int l = 0; l < L; ++l) p[l] /= s;
}

}  // namespace

extern "C" {

// Dense C^l(g) for keep mantissa bits (keep = 0: the base g^0), in fp64 (exact).
int mlmc_oracle_float_compress(const void* g, int dtype, int64_t d, int keep, double* out) {
    if (d < 1 || keep < 0 || keep > float_mantissa_bits(dtype)) return ORA_ERR_ARG;
    if (int rc = check_finite(g, dtype, d)) return rc;
    for (int64_t i = 0; i < d; ++i) out[i] = float_truncate(elem(g, dtype, i), keep);
    return ORA_OK;
}

// One worker's floating-point MLMC message and (optionally) its dense estimate.
//   expo_out[d]: biased exponent field of every entry.  planes_out: (1 + w_max) planes of ceil(d/32) words,
//   plane 0 = raw sign bits, plane j (1..w_l) = bit (w_l - j) of the level's mantissa field
//   f = mantissa digits mb_{l-1}+1 .. mb_l read as an integer;  est_out[d] = g^0 + (C^l - C^{l-1}) / p_l.
int mlmc_oracle_floatbits(const void* g, int dtype, int64_t d, const int32_t* mb, int L, const double* p_in,
                          uint64_t seed, uint64_t step, uint64_t worker, int force_level,
                          double* p_out, int32_t* level_out, double* p_sel_out, double* u_out, double* margin_out,
                          uint8_t* expo_out, uint32_t* planes_out, int32_t w_max, double* est_out) {
    if (d < 1 || !level_out || !p_sel_out) return ORA_ERR_ARG;
    const int F = float_mantissa_bits(dtype);
    if (int rc = check_mantissa_schedule(mb, L, F)) return rc;
    if (int rc = check_finite(g, dtype, d)) return rc;
    std::vector<double> p(static_cast<size_t>(L));
    if (p_in) {
        if (int rc = normalise_fixed(p_in, L, p.data())) return rc;
    } else {
        float_default_probs(mb, L, p.data());
    }
    const double u = uniform01(seed, step, worker);
    int level;
    double margin;
    draw_level(p.data(), L, u, &level, &margin);
    if (force_level >= 0) {
        if (force_level >= L) return ORA_ERR_ARG;
        level = force_level;
    }
    const double p_sel = p[static_cast<size_t>(level)];
    if (p_out) std::copy(p.begin(), p.end(), p_out);
    if (u_out) *u_out = u;
    if (margin_out) *margin_out = margin;
    *level_out = level;
    *p_sel_out = p_sel;
    const int lo = level ? mb[level - 1] : 0, hi = mb[level], w = hi - lo;
    const int64_t words = (d + 31) / 32;
    if (planes_out) {
        if (w > w_max) return ORA_ERR_CAPACITY;
        std::fill(planes_out, planes_out + (1 + w) * words, 0u);
    }
    for (int64_t i = 0; i < d; ++i) {
        const float x = elem(g, dtype, i);
        uint32_t bits;
        std::memcpy(&bits, &x, sizeof bits);
        if (expo_out) expo_out[i] = static_cast<uint8_t>((bits >> 23) & 0xFFu);
        if (planes_out) {
            const int64_t wd = i >> 5;
            const uint32_t bit = 1u << (i & 31);
            if (bits >> 31) planes_out[wd] |= bit;
            // mantissa digit j (1-based from the most significant) is bit 23 - j of the fp32 encoding
            for (int j = 1; j <= w; ++j)
                if ((bits >> (23 - (lo + j))) & 1u) planes_out[j * words + wd] |= bit;
        }
        if (est_out) {
            const double base = float_truncate(x, 0);
            const double res = float_truncate(x, hi) - float_truncate(x, lo);
            est_out[i] = base + res / p_sel;
        }
    }
    return ORA_OK;
}

// Decode a floating-point message into the dense estimate (fp64).
int mlmc_oracle_floatbits_decode(const uint8_t* expo, const uint32_t* planes, int64_t d, int dtype, const int32_t* mb,
                                 int L, int level, double p_sel, double* est_out) {
    if (level < 0 || level >= L || d < 1) return ORA_ERR_ARG;
    (void)dtype;
    const int lo = level ? mb[level - 1] : 0, hi = mb[level], w = hi - lo;
    const int64_t words = (d + 31) / 32;
    for (int64_t i = 0; i < d; ++i) {
        const int64_t wd = i >> 5;
        const int t = static_cast<int>(i & 31);
        uint32_t f = 0;
        for (int j = 1; j <= w; ++j) f = (f << 1) | ((planes[j * words + wd] >> t) & 1u);
        const int E = expo[i];
        // exponent field 0: no leading one, and the scale of exponent field 1
        const double base = E ? std::ldexp(1.0, E - 127) : 0.0;
        const double unit = std::ldexp(1.0, (E ? E : 1) - 127 - hi);
        const double v = base + static_cast<double>(f) * unit / p_sel;
        est_out[i] = ((planes[wd] >> t) & 1u) ? -v : v;
    }
    return ORA_OK;
}

// Server average of M dense estimates given as fp64 rows (used for the floating-point and RTN messages, whose
// decoded form is dense): out = (1/M) sum_m est_m, scale = (1/M) sum_m |est_m|.
int mlmc_oracle_aggregate_dense(int M, const double* const* est, int64_t d, double* out, double* scale_out) {
    if (M < 1 || d < 1) return ORA_ERR_ARG;
    std::fill(out, out + d, 0.0);
    if (scale_out) std::fill(scale_out, scale_out + d, 0.0);
    for (int m = 0; m < M; ++m)
        for (int64_t i = 0; i < d; ++i) {
            out[i] += est[m][i];
            if (scale_out) scale_out[i] += std::fabs(est[m][i]);
        }
    const double inv = 1.0 / static_cast<double>(M);
    for (int64_t i = 0; i < d; ++i) {
        out[i] *= inv;
        if (scale_out) scale_out[i] *= inv;
    }
    return ORA_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// s-Top-k (Sec. 2.2 "s-segmented Top-k", App. D)
// ---------------------------------------------------------------------------------------------
// The vector is sorted by magnitude and cut into segments of length s (the last one may be shorter);
// level l keeps the l + 1 segments of largest norm.  Sorted by magnitude, segment norms are
// non-increasing, so these are the first l + 1 segments: C^l = Top-(s (l + 1)), L = ceil(d / s) levels,
// and the residual of level l is the l-th segment (Sec. 3.2, remark on the residual).
extern "C" int mlmc_oracle_stopk(const void* g, int dtype, int64_t d, int64_t s, const double* p_in,
                                 uint64_t seed, uint64_t step, uint64_t worker, int force_level,
                                 double* p_out, double* delta_out, int32_t* level_out, double* p_sel_out,
                                 double* u_out, double* margin_out,
                                 int64_t* count_out, uint32_t* idx_out, float* val_out, int64_t capacity) {
    if (d < 1 || s < 1) return ORA_ERR_ARG;
    const int64_t L = (d + s - 1) / s;
    if (L > (int64_t(1) << 24)) return ORA_ERR_ARG;
    std::vector<int64_t> k(static_cast<size_t>(L));
    for (int64_t l = 0; l < L; ++l) k[static_cast<size_t>(l)] = std::min(d, s * (l + 1));
    return mlmc_oracle_topk(g, dtype, d, k.data(), static_cast<int>(L), p_in, seed, step, worker, force_level,
                            p_out, delta_out, level_out, p_sel_out, u_out, margin_out, count_out, idx_out, val_out,
                            capacity);
}

// ---------------------------------------------------------------------------------------------
// MLMC-RTN (Sec. 3.2 end, App. G)
// ---------------------------------------------------------------------------------------------
// C^l(v) = clip(delta^l round(v / delta^l), -c, c),  delta^l = 2c / (2^{r_l} - 1),  c = max_i |v_i|,
// for the bit widths r_0 < ... < r_{L-2} <= 16; level L-1 is the identity (Def. 3.1).  C^{-1} = 0.
// The rounding decides an integer, so its arithmetic is fixed: with inv = fl32((2^r - 1) / (2c)) and
// delta = fl32(2c / (2^r - 1)) (each the fp64 quotient rounded once to fp32),
//   t = fl32(v * inv),  k = t rounded to the nearest integer, ties to even,  C = clip(fl32(k * delta), -c, c).
// Residuals, their norms, the probabilities and the scaling by 1/p are fp64.
namespace {

int check_rtn_schedule(const int32_t* r, int L) {
    if (L < 1) return ORA_ERR_ARG;
    int prev = 0;
    for (int l = 0; l + 1 < L; ++l) {
        if (r[l] <= prev || r[l] > 16) return ORA_ERR_SCHEDULE;
        prev = r[l];
    }
    return ORA_OK;
}

float rtn_value(float v, float c, int r) {
    if (!(c > 0.0f)) return 0.0f;
    const double steps = static_cast<double>((1u << r) - 1u);
    const float inv = static_cast<float>(steps / (2.0 * static_cast<double>(c)));
    const float delta = static_cast<float>(2.0 * static_cast<double>(c) / steps);
    const float t = v * inv;
    const float k = std::nearbyintf(t);  // default rounding mode: to nearest, ties to even
    const float x = k * delta;
    return std::fmin(std::fmax(x, -c), c);
}

}  // namespace

extern "C" {

// Dense C^l(g) of one RTN level (level = L - 1: the identity), fp64 copies of the fp32 grid values.
int mlmc_oracle_rtn_compress(const void* g, int dtype, int64_t d, const int32_t* r, int L, int level, double* out) {
    if (d < 1 || level < 0 || level >= L) return ORA_ERR_ARG;
    if (int rc = check_rtn_schedule(r, L)) return rc;
    if (int rc = check_finite(g, dtype, d)) return rc;
    float c = 0.0f;
    for (int64_t i = 0; i < d; ++i) c = std::max(c, std::fabs(elem(g, dtype, i)));
    for (int64_t i = 0; i < d; ++i) {
        const float v = elem(g, dtype, i);
        out[i] = (level == L - 1) ? static_cast<double>(v) : static_cast<double>(rtn_value(v, c, r[level]));
    }
    return ORA_OK;
}

// One worker's MLMC-RTN message: val_out[d] = (float)((C^l - C^{l-1})_i / p_l), dense.
int mlmc_oracle_rtn(const void* g, int dtype, int64_t d, const int32_t* r, int L, const double* p_in,
                    uint64_t seed, uint64_t step, uint64_t worker, int force_level,
                    double* p_out, double* delta_out, int32_t* level_out, double* p_sel_out, double* u_out,
                    double* margin_out, float* c_out, float* val_out) {
    if (d < 1 || !level_out || !p_sel_out) return ORA_ERR_ARG;
    if (int rc = check_rtn_schedule(r, L)) return rc;
    if (int rc = check_finite(g, dtype, d)) return rc;
    std::vector<double> p(static_cast<size_t>(L)), delta(static_cast<size_t>(L));
    if (p_in)
        if (int rc = normalise_fixed(p_in, L, p.data())) return rc;
    float c = 0.0f;
    for (int64_t i = 0; i < d; ++i) c = std::max(c, std::fabs(elem(g, dtype, i)));
    auto level_value = [&](float v, int l) -> double {
        if (l < 0) return 0.0;
        if (l == L - 1) return static_cast<double>(v);
        return static_cast<double>(rtn_value(v, c, r[l]));
    };
    for (int l = 0; l < L; ++l) {
        double s2 = 0.0;
        for (int64_t i = 0; i < d; ++i) {
            const float v = elem(g, dtype, i);
            const double res = level_value(v, l) - level_value(v, l - 1);
            s2 += res * res;
        }
        delta[static_cast<size_t>(l)] = std::sqrt(s2);
    }
    if (!p_in) adaptive_probs(delta.data(), L, p.data());
    const double u = uniform01(seed, step, worker);
    int level;
    double margin;
    draw_level(p.data(), L, u, &level, &margin);
    if (force_level >= 0) {
        if (force_level >= L) return ORA_ERR_ARG;
        level = force_level;
    }
    const double p_sel = p[static_cast<size_t>(level)];
    if (p_out) std::copy(p.begin(), p.end(), p_out);
    if (delta_out) std::copy(delta.begin(), delta.end(), delta_out);
    if (u_out) *u_out = u;
    if (margin_out) *margin_out = margin;
    if (c_out) *c_out = c;
    *level_out = level;
    *p_sel_out = p_sel;
    if (val_out)
        for (int64_t i = 0; i < d; ++i) {
            const float v = elem(g, dtype, i);
            const double res = level_value(v, level) - level_value(v, level - 1);
            val_out[i] = (p_sel > 0.0) ? static_cast<float>(res / p_sel) : 0.0f;
        }
    return ORA_OK;
}

}  // extern "C"
