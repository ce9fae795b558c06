// C ABI of the MLMC compression library: context, argument checks and the launch sequences.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

using namespace mlmc;

struct mlmc_ctx {
    Workspace ws;
    void* slab;
    size_t slab_bytes;
};

namespace {

struct SlabPlanner {
    size_t off = 0;
    size_t take(size_t bytes) {
        const size_t at = off;
        off += (bytes + 255) & ~size_t(255);
        return at;
    }
};

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

int check_common(const mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, int L) {
    if (!ctx || !g) return MLMC_ERR_ARG;
    if (dtype != MLMC_F32 && dtype != MLMC_BF16) return MLMC_ERR_ARG;
    if (d < 1 || d > ctx->ws.d_max || d >= (int64_t(1) << 32)) return MLMC_ERR_ARG;
    if (M < 1 || M > ctx->ws.M_max) return MLMC_ERR_ARG;
    if (L < 1 || L > ctx->ws.L_max) return MLMC_ERR_ARG;
    if (ld < d) return MLMC_ERR_ARG;
    const int64_t esize = (dtype == MLMC_BF16) ? 2 : 4;
    if (reinterpret_cast<uintptr_t>(g) % 16 != 0) return MLMC_ERR_ARG;
    if (M > 1 && (ld * esize) % 16 != 0) return MLMC_ERR_ARG;
    return MLMC_OK;
}

int check_topk_schedule(const int64_t* k, int L, int64_t d) {
    if (!k) return MLMC_ERR_ARG;
    int64_t prev = 0;
    for (int l = 0; l < L; ++l) {
        if (k[l] < prev || k[l] > d) return MLMC_ERR_SCHEDULE;
        prev = k[l];
    }
    return k[L - 1] == d ? MLMC_OK : MLMC_ERR_SCHEDULE;  // Def. 3.1: the top level is the identity
}

template <typename I>
int check_bit_schedule(const I* b, int L, int32_t* b32) {
    if (!b) return MLMC_ERR_ARG;
    int64_t prev = 0;
    for (int l = 0; l < L; ++l) {
        if (b[l] <= prev || b[l] > 23) return MLMC_ERR_SCHEDULE;
        prev = b[l];
        b32[l] = (int32_t)b[l];
    }
    return MLMC_OK;
}

// RTN widths r_0 < ... < r_{L-2} <= 16 (App. G); level L-1 is the identity and has no width.
template <typename I>
int check_rtn_schedule(const I* r, int L, int32_t* r32) {
    if (L < 1 || L > 17) return MLMC_ERR_ARG;
    if (L > 1 && !r) return MLMC_ERR_ARG;
    int64_t prev = 0;
    for (int l = 0; l + 1 < L; ++l) {
        if (r[l] <= prev || r[l] > 16) return MLMC_ERR_SCHEDULE;
        prev = r[l];
        r32[l] = (int32_t)r[l];
    }
    return MLMC_OK;
}

// Mantissa digits mb_0 < ... < mb_{L-1} = F kept by the floating-point levels (App. B); the top level is the identity.
int check_mantissa_schedule(const int32_t* mb, int L, int F) {
    if (!mb) return MLMC_ERR_ARG;
    int prev = 0;
    for (int l = 0; l < L; ++l) {
        if (mb[l] <= prev || mb[l] > F) return MLMC_ERR_SCHEDULE;
        prev = mb[l];
    }
    return mb[L - 1] == F ? MLMC_OK : MLMC_ERR_SCHEDULE;
}

// Lemma 3.2 asks for non-zero probabilities; they are renormalised in fp64.
int normalise_probs(const double* p, int L, double* out) {
    double s = 0.0;
    for (int l = 0; l < L; ++l) {
        if (!(p[l] > 0.0) || !std::isfinite(p[l])) return MLMC_ERR_PROB;
        s += p[l];
    }
    if (std::fabs(s - 1.0) > 1e-9) return MLMC_ERR_PROB;
    for (int l = 0; l < L; ++l) out[l] = p[l] / s;
    return MLMC_OK;
}

int finish(cudaError_t e) { return e == cudaSuccess ? MLMC_OK : MLMC_ERR_CUDA; }

// Thresholds of every live query (sweep 1 + the two masked digit passes for fp32).
// sweep 1 (leading-digit histogram), and for fp32 sweep 2 (candidates [+ energies]) and the two remaining
// digit passes over the candidates.
// brackets (fixed p, fp32): the first sweep also collects the keys of the bins around last call's boundary bins;
// where both boundary bins of a worker's band fall inside, the candidate sweep has nothing left to do.
void run_selection(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, int L, bool sums,
                   bool brackets, cudaStream_t s) {
    brackets = brackets && dtype == MLMC_F32 && !sums && L > 1;
    launch_reset_selection(ws, dtype, d, M, s);
    launch_hist1(ws, g, dtype, d, M, ld, brackets, s);
    launch_resolve1(ws, dtype, M, L, brackets, s);
    if (dtype == MLMC_F32) {
        launch_sums_candidates(ws, g, d, M, ld, L, sums, brackets, s);
        if (L > 1) {
            launch_digit_pass(ws, g, d, M, ld, 2, s);
            launch_resolve23(ws, M, L, 2, s);
            launch_digit_pass(ws, g, d, M, ld, 3, s);
            launch_resolve23(ws, M, L, 3, s);
        }
    }
}

void run_band_norms(Workspace& ws, const void* g, int dtype, int64_t d, int M, int64_t ld, int L, cudaStream_t s) {
    if (dtype == MLMC_BF16)
        launch_norm_from_hist_bf16(ws, M, L, s);
    else
        launch_band_norms_fp32(ws, g, d, M, ld, L, s);
}

}  // namespace

extern "C" {

int mlmc_create(mlmc_ctx** out, int device, int64_t d_max, int M_max, int L_max) {
    if (!out || d_max < 1 || d_max >= (int64_t(1) << 32) || M_max < 1 || M_max > kEmitMaxWorkers || L_max < 1 ||
        L_max > kMaxLevels)
        return MLMC_ERR_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return MLMC_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MLMC_ERR_CUDA;
    if (configure_select_kernels() != MLMC_OK || configure_emit_kernels() != MLMC_OK ||
        configure_bit_kernels() != MLMC_OK || configure_sort_kernels() != MLMC_OK)
        return MLMC_ERR_CUDA;

    mlmc_ctx* ctx = new (std::nothrow) mlmc_ctx();
    if (!ctx) return MLMC_ERR_NOMEM;
    Workspace& ws = ctx->ws;
    ws.device = device;
    ws.d_max = d_max;
    ws.M_max = M_max;
    ws.L_max = L_max;
    ws.sm_count = prop.multiProcessorCount;
    ws.launches = 0;
    ws.timing = false;
    ws.last_emit_tiles = 0;
    ws.timing_used = 0;
    ws.ev_start = ws.ev_stop = nullptr;
    ws.ev_id = nullptr;
    for (int i = 0; i < K_COUNT; ++i) ws.launches_by_id[i] = 0;
    ws.norm_ctas = ws.sm_count * 4;
    ws.sum_ctas = ws.sm_count * 4;
    ws.cur_norm_ctas = ws.cur_sum_ctas = 0;
    // candidate keys: a quarter of the row (boundary bins normally hold a few percent of it); small rows fit whole
    ws.cand_cap = d_max / 4 > (int64_t(1) << 20) ? d_max / 4 : (d_max < (int64_t(1) << 20) ? d_max : (int64_t(1) << 20));
    ws.stat_ctas = ws.sm_count * 4;
    ws.cur_stat_ctas = 0;
    const int64_t emit_tiles = (d_max + kEmitTile - 1) / kEmitTile;
    const int64_t agg_tiles = (d_max + kAggTile - 1) / kAggTile;
    ws.max_tiles = emit_tiles * M_max;

    SlabPlanner pl;
    const size_t o_status = pl.take(sizeof(int));
    const size_t o_werr = pl.take(sizeof(int) * M_max);
    const size_t o_hist1 = pl.take(sizeof(uint32_t) * kBins1 * M_max);
    const size_t o_table1 = pl.take((size_t)kBins1 * M_max);
    const size_t o_hist2 = pl.take(sizeof(uint32_t) * kMaxQueries * kBins23 * M_max);
    const size_t o_map2 = pl.take((size_t)kMaxQueries * kBins23 * M_max);
    const size_t o_hist3 = pl.take(sizeof(uint32_t) * kMaxQueries * kBins23 * M_max);
    const size_t o_queries = pl.take(sizeof(Query) * kMaxQueries * M_max);
    const size_t o_band = pl.take(sizeof(double) * kMaxLevels * ws.norm_ctas * M_max);
    const size_t o_sum = pl.take(sizeof(double) * kMaxLevels * ws.sum_ctas * M_max);
    const size_t o_cpart = pl.take(sizeof(unsigned long long) * kMaxLevels * 4 * M_max);
    const size_t o_ckeys = pl.take(sizeof(uint32_t) * ws.cand_cap * M_max);
    const size_t o_ccount = pl.take(sizeof(uint32_t) * M_max);
    const size_t o_cover = pl.take(sizeof(int) * M_max);
    const size_t o_k = pl.take(sizeof(int64_t) * kMaxLevels);
    const size_t o_pfix = pl.take(sizeof(double) * kMaxLevels);
    const size_t o_pall = pl.take(sizeof(double) * kMaxLevels * M_max);
    const size_t o_dall = pl.take(sizeof(double) * kMaxLevels * M_max);
    const size_t o_u = pl.take(sizeof(double) * M_max);
    const size_t o_emit = pl.take(sizeof(EmitParams) * M_max);
    const size_t o_tdesc = pl.take(sizeof(uint4) * ws.max_tiles);
    const size_t o_tmax = pl.take(sizeof(uint32_t) * ws.max_tiles * kEmitGroups);
    const size_t o_groupn = pl.take(sizeof(uint32_t) * M_max);
    const size_t o_wtiles = pl.take(sizeof(uint32_t) * ws.max_tiles);
    const size_t o_tilen = pl.take(sizeof(uint32_t) * M_max);
    const size_t o_cfloor = pl.take(sizeof(uint32_t) * M_max);
    const size_t o_aggoff = pl.take(sizeof(uint32_t) * (agg_tiles + 1) * M_max);
    const size_t o_gmax = pl.take(sizeof(uint32_t) * M_max);
    const size_t o_S = pl.take(sizeof(unsigned long long) * kMaxLevels * ws.stat_ctas * M_max);
    const size_t o_blevel = pl.take(sizeof(int32_t) * M_max);
    ws.big_cap = d_max < (int64_t(1) << 20) ? d_max : (int64_t(1) << 20);
    const size_t o_pbig = pl.take(sizeof(double) * ws.big_cap);
    const size_t o_cbig = pl.take(sizeof(double) * ws.big_cap);
    ws.rtn_ctas = ws.sm_count * 8;
    ws.cur_rtn_ctas = 0;
    const size_t o_rtn = pl.take(sizeof(double) * kMaxLevels * ws.rtn_ctas * M_max);
    const size_t o_pbin = pl.take(sizeof(uint32_t) * kMaxLevels * M_max);
    const size_t o_brk = pl.take(sizeof(uint4) * M_max);
    const size_t o_bhit = pl.take(sizeof(int) * M_max);
    const size_t o_bstat = pl.take(sizeof(unsigned long long) * 4);
    ws.sort_scratch = nullptr;
    ws.sort_rows = 0;
    ws.sig_d = ws.sig_ld = -1;
    ws.sig_M = ws.sig_L = ws.sig_dtype = -1;

    ctx->slab_bytes = pl.off;
    if (cudaMalloc(&ctx->slab, ctx->slab_bytes) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return MLMC_ERR_NOMEM;
    }
    if (cudaMemset(ctx->slab, 0, ctx->slab_bytes) != cudaSuccess) {
        cudaFree(ctx->slab);
        delete ctx;
        return MLMC_ERR_CUDA;
    }
    char* base = static_cast<char*>(ctx->slab);
    ws.status = reinterpret_cast<int*>(base + o_status);
    ws.worker_err = reinterpret_cast<int*>(base + o_werr);
    ws.hist1 = reinterpret_cast<uint32_t*>(base + o_hist1);
    ws.table1 = reinterpret_cast<uint8_t*>(base + o_table1);
    ws.hist2 = reinterpret_cast<uint32_t*>(base + o_hist2);
    ws.map2 = reinterpret_cast<uint8_t*>(base + o_map2);
    ws.hist3 = reinterpret_cast<uint32_t*>(base + o_hist3);
    ws.queries = reinterpret_cast<Query*>(base + o_queries);
    ws.band_partial = reinterpret_cast<double*>(base + o_band);
    ws.sum_partial = reinterpret_cast<double*>(base + o_sum);
    ws.cand_S = reinterpret_cast<unsigned long long*>(base + o_cpart);
    ws.cand_keys = reinterpret_cast<uint32_t*>(base + o_ckeys);
    ws.cand_count = reinterpret_cast<uint32_t*>(base + o_ccount);
    ws.cand_overflow = reinterpret_cast<int*>(base + o_cover);
    ws.k_dev = reinterpret_cast<int64_t*>(base + o_k);
    ws.p_fixed = reinterpret_cast<double*>(base + o_pfix);
    ws.p_all = reinterpret_cast<double*>(base + o_pall);
    ws.delta_all = reinterpret_cast<double*>(base + o_dall);
    ws.u_dev = reinterpret_cast<double*>(base + o_u);
    ws.emit = reinterpret_cast<EmitParams*>(base + o_emit);
    ws.tile_desc = reinterpret_cast<uint4*>(base + o_tdesc);
    ws.tile_max = reinterpret_cast<uint32_t*>(base + o_tmax);
    ws.worker_tiles = reinterpret_cast<uint32_t*>(base + o_wtiles);
    ws.tile_n = reinterpret_cast<uint32_t*>(base + o_tilen);
    ws.group_n = reinterpret_cast<uint32_t*>(base + o_groupn);
    ws.cand_floor = reinterpret_cast<uint32_t*>(base + o_cfloor);
    ws.agg_offsets = reinterpret_cast<uint32_t*>(base + o_aggoff);
    ws.gmax_bits = reinterpret_cast<uint32_t*>(base + o_gmax);
    ws.S_partial = reinterpret_cast<unsigned long long*>(base + o_S);
    ws.bit_level = reinterpret_cast<int32_t*>(base + o_blevel);
    ws.p_big = reinterpret_cast<double*>(base + o_pbig);
    ws.cdf_big = reinterpret_cast<double*>(base + o_cbig);
    ws.rtn_partial = reinterpret_cast<double*>(base + o_rtn);
    ws.prev_bin = reinterpret_cast<uint32_t*>(base + o_pbin);
    ws.bracket = reinterpret_cast<uint4*>(base + o_brk);
    ws.bracket_hit = reinterpret_cast<int*>(base + o_bhit);
    ws.bracket_stats = reinterpret_cast<unsigned long long*>(base + o_bstat);
    cudaMemset(ws.prev_bin, 0xFF, sizeof(uint32_t) * kMaxLevels * M_max);
    if (cudaDeviceSynchronize() != cudaSuccess) {
        cudaFree(ctx->slab);
        delete ctx;
        return MLMC_ERR_CUDA;
    }
    *out = ctx;
    return MLMC_OK;
}

int mlmc_destroy(mlmc_ctx* ctx) {
    if (!ctx) return MLMC_ERR_ARG;
    DeviceGuard guard(ctx->ws.device);
    cudaDeviceSynchronize();
    if (ctx->ws.ev_start) {
        for (int i = 0; i < kTimingPool; ++i) {
            cudaEventDestroy(ctx->ws.ev_start[i]);
            cudaEventDestroy(ctx->ws.ev_stop[i]);
        }
        delete[] ctx->ws.ev_start;
        delete[] ctx->ws.ev_stop;
        delete[] ctx->ws.ev_id;
    }
    if (ctx->ws.sort_scratch) cudaFree(ctx->ws.sort_scratch);
    const cudaError_t e = cudaFree(ctx->slab);
    delete ctx;
    return finish(e);
}

int mlmc_get_status(mlmc_ctx* ctx, void* stream) {
    if (!ctx) return MLMC_ERR_ARG;
    DeviceGuard guard(ctx->ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st = 0;
    if (cudaMemcpyAsync(&st, ctx->ws.status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return MLMC_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MLMC_ERR_CUDA;
    if (st != 0) {
        if (cudaMemsetAsync(ctx->ws.status, 0, sizeof(int), s) != cudaSuccess) return MLMC_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return MLMC_ERR_CUDA;
    }
    return st;
}

int64_t mlmc_launch_count(const mlmc_ctx* ctx) { return ctx ? ctx->ws.launches : 0; }

static const char* const kKernelNames[K_COUNT] = {
    "draw_fixed", "init_queries", "uniforms", "hist1", "resolve1", "sums_candidates", "cand_pass2", "masked_pass2",
    "resolve2", "cand_pass3", "masked_pass3", "resolve3", "cand_sums", "norm_sweep", "norm_from_hist_bf16", "probs_draw", "copy_probs", "emit", "agg_offsets",
    "aggregate_topk", "absmax", "bit_stats", "bit_probs_draw", "bit_pack", "aggregate_bitwise", "tile_list", "band_count", "band_scan", "bit_pack_wide", "reset",
    "float_draw", "float_pack", "aggregate_floatbits", "rtn_stats", "rtn_probs_draw", "rtn_emit", "aggregate_dense", "stopk_draw", "stopk_params",
    "sort_count", "sort_scan", "sort_scatter", "segment_norms"};

int mlmc_kernel_count(void) { return K_COUNT; }

const char* mlmc_kernel_name(int id) { return (id >= 0 && id < K_COUNT) ? kKernelNames[id] : ""; }

int mlmc_timing_enable(mlmc_ctx* ctx, int on) {
    if (!ctx) return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    DeviceGuard guard(ws.device);
    if (on && !ws.ev_start) {
        ws.ev_start = new (std::nothrow) cudaEvent_t[kTimingPool];
        ws.ev_stop = new (std::nothrow) cudaEvent_t[kTimingPool];
        ws.ev_id = new (std::nothrow) int[kTimingPool];
        if (!ws.ev_start || !ws.ev_stop || !ws.ev_id) return MLMC_ERR_NOMEM;
        for (int i = 0; i < kTimingPool; ++i)
            if (cudaEventCreate(&ws.ev_start[i]) != cudaSuccess || cudaEventCreate(&ws.ev_stop[i]) != cudaSuccess)
                return MLMC_ERR_CUDA;
    }
    ws.timing = on != 0;
    ws.timing_used = 0;
    return MLMC_OK;
}

int mlmc_timing_read(mlmc_ctx* ctx, double* total_ms, int64_t* launches, void* stream) {
    if (!ctx || !total_ms || !launches) return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    DeviceGuard guard(ws.device);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MLMC_ERR_CUDA;
    for (int i = 0; i < K_COUNT; ++i) {
        total_ms[i] = 0.0;
        launches[i] = 0;
    }
    for (int i = 0; i < ws.timing_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ws.ev_start[i], ws.ev_stop[i]) != cudaSuccess) return MLMC_ERR_CUDA;
        total_ms[ws.ev_id[i]] += ms;
        launches[ws.ev_id[i]]++;
    }
    ws.timing_used = 0;
    return MLMC_OK;
}

int mlmc_read_u(mlmc_ctx* ctx, uint64_t seed, uint64_t step, int M, double* u_host, void* stream) {
    if (!ctx || !u_host || M < 1 || M > ctx->ws.M_max) return MLMC_ERR_ARG;
    DeviceGuard guard(ctx->ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    launch_uniforms(ctx->ws, M, seed, step, s);
    if (cudaMemcpyAsync(u_host, ctx->ws.u_dev, sizeof(double) * M, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return finish(cudaStreamSynchronize(s));
}

int mlmc_read_bracket_stats(mlmc_ctx* ctx, uint64_t* stats_host, void* stream) {
    if (!ctx || !stats_host) return MLMC_ERR_ARG;
    DeviceGuard guard(ctx->ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(stats_host, ctx->ws.bracket_stats, sizeof(uint64_t) * 3, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return finish(cudaStreamSynchronize(s));
}

int mlmc_read_listed_tiles(mlmc_ctx* ctx, int M, uint32_t* listed_host, int64_t* tiles_host, void* stream) {
    if (!ctx || !listed_host || !tiles_host || M < 1 || M > ctx->ws.M_max) return MLMC_ERR_ARG;
    DeviceGuard guard(ctx->ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    *tiles_host = ctx->ws.last_emit_tiles * kEmitGroups;
    if (cudaMemcpyAsync(listed_host, ctx->ws.group_n, sizeof(uint32_t) * M, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return MLMC_ERR_CUDA;
    return finish(cudaStreamSynchronize(s));
}

int mlmc_level_probs(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, int kind,
                     const int64_t* sched, int L, const double* p_host, double* p_out, double* delta_out,
                     void* stream) {
    if (int rc = check_common(ctx, g, dtype, d, M, ld, L)) return rc;
    if (!p_out || (kind != MLMC_TOPK && kind != MLMC_BITWISE && kind != MLMC_RTN)) return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    double pn[kMaxLevels];
    int32_t b32[kMaxLevels];
    if (kind == MLMC_TOPK) {
        if (int rc = check_topk_schedule(sched, L, d)) return rc;
    } else if (kind == MLMC_BITWISE) {
        if (int rc = check_bit_schedule(sched, L, b32)) return rc;
    } else {
        if (int rc = check_rtn_schedule(sched, L, b32)) return rc;
    }
    if (p_host)
        if (int rc = normalise_probs(p_host, L, pn)) return rc;
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
    if (p_host) cudaMemcpyAsync(ws.p_fixed, pn, sizeof(double) * L, cudaMemcpyHostToDevice, s);
    const bool need_data = (p_host == nullptr) || (delta_out != nullptr);
    if (kind == MLMC_TOPK) {
        cudaMemcpyAsync(ws.k_dev, sched, sizeof(int64_t) * L, cudaMemcpyHostToDevice, s);
        if (need_data) {
            launch_init_queries_adaptive(ws, M, L, d, s);
            run_selection(ws, g, dtype, d, M, ld, L, true, false, s);
            run_band_norms(ws, g, dtype, d, M, ld, L, s);
            launch_probs_draw(ws, dtype, M, L, d, true, false, 0, 0, nullptr, s);
        }
    } else if (kind == MLMC_BITWISE) {
        if (need_data) {
            launch_absmax(ws, g, dtype, d, M, ld, s);
            launch_bit_stats(ws, g, dtype, d, M, ld, b32, L, s);
            launch_bit_probs_draw(ws, M, b32, L, true, true, 0, 0, nullptr, s);
        }
    } else {
        if (need_data) {
            launch_absmax(ws, g, dtype, d, M, ld, s);
            launch_rtn_stats(ws, g, dtype, d, M, ld, b32, L, s);
            launch_rtn_probs_draw(ws, M, L, true, true, 0, 0, nullptr, s);
        }
    }
    launch_copy_probs(ws, M, L, p_host ? ws.p_fixed : nullptr, p_out, delta_out, s);
    return finish(cudaGetLastError());
}

int mlmc_compress_topk(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, const int64_t* k,
                       int L, const double* p, uint64_t seed, uint64_t step, const mlmc_topk_msgs* out,
                       void* stream) {
    if (int rc = check_common(ctx, g, dtype, d, M, ld, L)) return rc;
    if (!out || !out->idx || !out->val || !out->count || !out->level || !out->p_sel || out->capacity < 0)
        return MLMC_ERR_ARG;
    if (int rc = check_topk_schedule(k, L, d)) return rc;
    double pn[kMaxLevels];
    if (p)
        if (int rc = normalise_probs(p, L, pn)) return rc;
    Workspace& ws = ctx->ws;
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
    cudaMemcpyAsync(ws.k_dev, k, sizeof(int64_t) * L, cudaMemcpyHostToDevice, s);
    const bool adaptive = (p == nullptr);
    if (adaptive) {
        launch_init_queries_adaptive(ws, M, L, d, s);
    } else {
        cudaMemcpyAsync(ws.p_fixed, pn, sizeof(double) * L, cudaMemcpyHostToDevice, s);
        // the bins stored by earlier calls belong to one problem: another shape or schedule starts afresh
        bool same = ws.sig_d == d && ws.sig_ld == ld && ws.sig_M == M && ws.sig_L == L && ws.sig_dtype == dtype;
        for (int l = 0; same && l < L; ++l) same = ws.sig_k[l] == k[l];
        if (!same) {
            cudaMemsetAsync(ws.prev_bin, 0xFF, sizeof(uint32_t) * kMaxLevels * ws.M_max, s);
            ws.sig_d = d; ws.sig_ld = ld; ws.sig_M = M; ws.sig_L = L; ws.sig_dtype = dtype;
            for (int l = 0; l < L; ++l) ws.sig_k[l] = k[l];
        }
        launch_draw_fixed(ws, M, L, d, seed, step, true, s);  // the draw does not depend on the data: only two thresholds are needed
    }
    run_selection(ws, g, dtype, d, M, ld, L, adaptive, !adaptive, s);
    if (adaptive) run_band_norms(ws, g, dtype, d, M, ld, L, s);
    launch_probs_draw(ws, dtype, M, L, d, adaptive, true, seed, step, out, s);
    launch_emit(ws, g, dtype, d, M, ld, *out, s);
    return finish(cudaGetLastError());
}

int mlmc_compress_bitwise(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* b,
                          int L, const double* p, uint64_t seed, uint64_t step, const mlmc_bit_msgs* out,
                          void* stream) {
    if (int rc = check_common(ctx, g, dtype, d, M, ld, L)) return rc;
    if (!out || !out->planes || !out->gmax || !out->level || !out->p_sel || out->w_max < 1) return MLMC_ERR_ARG;
    int32_t b32[kMaxLevels];
    if (int rc = check_bit_schedule(b, L, b32)) return rc;
    double pn[kMaxLevels];
    if (p)
        if (int rc = normalise_probs(p, L, pn)) return rc;
    Workspace& ws = ctx->ws;
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
    const bool adaptive = (p == nullptr);
    if (!adaptive) cudaMemcpyAsync(ws.p_fixed, pn, sizeof(double) * L, cudaMemcpyHostToDevice, s);
    launch_absmax(ws, g, dtype, d, M, ld, s);
    if (adaptive) launch_bit_stats(ws, g, dtype, d, M, ld, b32, L, s);
    launch_bit_probs_draw(ws, M, b32, L, adaptive, false, seed, step, out, s);
    launch_bit_pack(ws, g, dtype, d, M, ld, b32, L, *out, s);
    return finish(cudaGetLastError());
}

int mlmc_aggregate(mlmc_ctx* ctx, int kind, const void* msgs, const int32_t* b, int L, int M, int64_t d, float* out,
                   void* stream) {
    if (!ctx || !msgs || !out) return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    if (d < 1 || d > ws.d_max || M < 1 || M > ws.M_max) return MLMC_ERR_ARG;
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (kind == MLMC_TOPK) {
        const mlmc_topk_msgs* t = static_cast<const mlmc_topk_msgs*>(msgs);
        if (!t->idx || !t->val || !t->count || !t->level) return MLMC_ERR_ARG;
        launch_aggregate_topk(ws, *t, M, d, out, s);
    } else if (kind == MLMC_BITWISE) {
        const mlmc_bit_msgs* t = static_cast<const mlmc_bit_msgs*>(msgs);
        if (!t->planes || !t->gmax || !t->level || !t->p_sel || L < 1 || L > kMaxLevels) return MLMC_ERR_ARG;
        int32_t b32[kMaxLevels];
        if (int rc = check_bit_schedule(b, L, b32)) return rc;
        launch_aggregate_bitwise(ws, *t, b32, L, M, d, out, s);
    } else {
        return MLMC_ERR_ARG;
    }
    return finish(cudaGetLastError());
}

int mlmc_compress_stopk(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, int64_t s_len,
                        const double* p, uint64_t seed, uint64_t step, const mlmc_topk_msgs* out, void* stream) {
    if (!ctx || s_len < 1 || d < 1) return MLMC_ERR_ARG;
    const int64_t L = (d + s_len - 1) / s_len;
    if (L <= kMaxLevels) {  // few segments: the general Top-k path with the uniform schedule k_l = min(d, s (l + 1))
        int64_t k[kMaxLevels];
        for (int64_t l = 0; l < L; ++l) k[l] = (s_len * (l + 1) < d) ? s_len * (l + 1) : d;
        return mlmc_compress_topk(ctx, g, dtype, d, M, ld, k, (int)L, p, seed, step, out, stream);
    }
    if (int rc = check_common(ctx, g, dtype, d, M, ld, 1)) return rc;
    if (!out || !out->idx || !out->val || !out->count || !out->level || !out->p_sel || out->capacity < 0)
        return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    if (L > ws.big_cap) return MLMC_ERR_ARG;
    if (!p) {
        // Adaptive p with many segments (Lemma 3.4 needs the norm of every segment): the rows are sorted, several
        // at a time, in scratch memory that the context allocates at the first such call.
        DeviceGuard guard(ws.device);
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        if (!ws.sort_scratch) {
            ws.sort_rows = stopk_sort_rows(ws.d_max, ws.big_cap, ws.M_max);
            if (cudaMalloc(&ws.sort_scratch, stopk_sort_scratch_bytes(ws.d_max, ws.big_cap, ws.M_max)) != cudaSuccess) {
                cudaGetLastError();
                ws.sort_scratch = nullptr;
                return MLMC_ERR_NOMEM;
            }
        }
        cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
        launch_reset_selection(ws, dtype, d, M, s);
        launch_hist1(ws, g, dtype, d, M, ld, false, s);  // the batch maxima for the emission, and the NaN / Inf check
        for (int m0 = 0; m0 < M; m0 += ws.sort_rows)
            launch_stopk_sorted_rows(ws, g, dtype, d, m0, (M - m0 < ws.sort_rows) ? M - m0 : ws.sort_rows, ld, s_len, L,
                                     seed, step, s);
        launch_stopk_params(ws, M, s_len, d, out, s);
        launch_emit(ws, g, dtype, d, M, ld, *out, s);
        return finish(cudaGetLastError());
    }
    // normalised p and its running sums in ascending l (the draw is min{ l : u < cdf_l }, the last cdf is 1)
    std::vector<double> pn((size_t)L), cdf((size_t)L);
    double sum = 0.0;
    for (int64_t l = 0; l < L; ++l) {
        if (!(p[l] > 0.0) || !std::isfinite(p[l])) return MLMC_ERR_PROB;
        sum += p[l];
    }
    if (std::fabs(sum - 1.0) > 1e-9) return MLMC_ERR_PROB;
    double c = 0.0;
    for (int64_t l = 0; l < L; ++l) {
        pn[(size_t)l] = p[l] / sum;
        c += pn[(size_t)l];
        cdf[(size_t)l] = (l == L - 1) ? 1.0 : c;
    }
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
    cudaMemcpyAsync(ws.p_big, pn.data(), sizeof(double) * L, cudaMemcpyHostToDevice, s);
    cudaMemcpyAsync(ws.cdf_big, cdf.data(), sizeof(double) * L, cudaMemcpyHostToDevice, s);
    if (cudaStreamSynchronize(s) != cudaSuccess) return MLMC_ERR_CUDA;  // the host arrays go out of scope below
    launch_stopk_draw(ws, M, L, s_len, d, seed, step, s);
    run_selection(ws, g, dtype, d, M, ld, 3, false, false, s);  // two queries per worker
    launch_stopk_params(ws, M, s_len, d, out, s);
    launch_emit(ws, g, dtype, d, M, ld, *out, s);
    return finish(cudaGetLastError());
}

int mlmc_compress_floatbits(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* mb,
                            int L, const double* p, uint64_t seed, uint64_t step, const mlmc_float_msgs* out,
                            void* stream) {
    if (int rc = check_common(ctx, g, dtype, d, M, ld, L)) return rc;
    if (!out || !out->expo || !out->planes || !out->level || !out->p_sel || out->w_max < 1) return MLMC_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(out->expo) % 16 != 0 || reinterpret_cast<uintptr_t>(out->planes) % 16 != 0)
        return MLMC_ERR_ARG;
    if (int rc = check_mantissa_schedule(mb, L, dtype == MLMC_BF16 ? 7 : 23)) return rc;
    double pn[kMaxLevels];
    if (p) {
        if (int rc = normalise_probs(p, L, pn)) return rc;
    } else {
        // App. B's lemma: p^l proportional to 2^-l for the unit schedule; for a general schedule its worst-case
        // argument gives p^l proportional to the largest residual of the level, 2^-mb_{l-1} - 2^-mb_l
        double sum = 0.0;
        for (int l = 0; l < L; ++l) {
            pn[l] = std::ldexp(1.0, -(l ? mb[l - 1] : 0)) - std::ldexp(1.0, -mb[l]);
            sum += pn[l];
        }
        for (int l = 0; l < L; ++l) pn[l] /= sum;
    }
    Workspace& ws = ctx->ws;
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
    cudaMemcpyAsync(ws.p_fixed, pn, sizeof(double) * L, cudaMemcpyHostToDevice, s);
    launch_compress_floatbits(ws, g, dtype, d, M, ld, mb, L, seed, step, *out, s);
    return finish(cudaGetLastError());
}

int mlmc_aggregate_floatbits(mlmc_ctx* ctx, const mlmc_float_msgs* msgs, const int32_t* mb, int L, int M, int64_t d,
                             float* out, void* stream) {
    if (!ctx || !msgs || !out || !msgs->expo || !msgs->planes || !msgs->level || !msgs->p_sel) return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    if (d < 1 || d > ws.d_max || M < 1 || M > ws.M_max || L < 1 || L > kMaxLevels) return MLMC_ERR_ARG;
    if (!mb) return MLMC_ERR_ARG;
    int prev = 0;
    for (int l = 0; l < L; ++l) {
        if (mb[l] <= prev || mb[l] > 23) return MLMC_ERR_SCHEDULE;
        prev = mb[l];
    }
    DeviceGuard guard(ws.device);
    launch_aggregate_floatbits(ws, *msgs, mb, L, M, d, out, static_cast<cudaStream_t>(stream));
    return finish(cudaGetLastError());
}

int mlmc_compress_rtn(mlmc_ctx* ctx, const void* g, int dtype, int64_t d, int M, int64_t ld, const int32_t* r, int L,
                      const double* p, uint64_t seed, uint64_t step, const mlmc_rtn_msgs* out, void* stream) {
    if (int rc = check_common(ctx, g, dtype, d, M, ld, L)) return rc;
    if (!out || !out->val || !out->c || !out->level || !out->p_sel || out->ldv < d) return MLMC_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(out->val) % 16 != 0) return MLMC_ERR_ARG;
    int32_t r32[kMaxLevels] = {};
    if (int rc = check_rtn_schedule(r, L, r32)) return rc;
    double pn[kMaxLevels];
    if (p)
        if (int rc = normalise_probs(p, L, pn)) return rc;
    Workspace& ws = ctx->ws;
    DeviceGuard guard(ws.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemsetAsync(ws.worker_err, 0, sizeof(int) * M, s);
    const bool adaptive = (p == nullptr);
    if (!adaptive) cudaMemcpyAsync(ws.p_fixed, pn, sizeof(double) * L, cudaMemcpyHostToDevice, s);
    launch_absmax(ws, g, dtype, d, M, ld, s);  // c = max |g|, and the NaN / Inf check
    if (adaptive) launch_rtn_stats(ws, g, dtype, d, M, ld, r32, L, s);
    launch_rtn_probs_draw(ws, M, L, adaptive, adaptive, seed, step, out, s);
    launch_rtn_emit(ws, g, dtype, d, M, ld, r32, L, *out, s);
    return finish(cudaGetLastError());
}

int mlmc_aggregate_rtn(mlmc_ctx* ctx, const mlmc_rtn_msgs* msgs, int M, int64_t d, float* out, void* stream) {
    if (!ctx || !msgs || !out || !msgs->val || !msgs->level || msgs->ldv < d) return MLMC_ERR_ARG;
    Workspace& ws = ctx->ws;
    if (d < 1 || d > ws.d_max || M < 1 || M > ws.M_max) return MLMC_ERR_ARG;
    DeviceGuard guard(ws.device);
    launch_aggregate_dense(ws, msgs->val, msgs->level, M, d, msgs->ldv, out, static_cast<cudaStream_t>(stream));
    return finish(cudaGetLastError());
}

}  // extern "C"
