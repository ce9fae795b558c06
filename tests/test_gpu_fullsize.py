"""Parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times.

The oracle cannot sort eight 124M-entry rows in reasonable time, so per workload and for the first and the last step
of the config
  * one worker's whole row goes through the oracle and is compared element by element
    (level, probability, every band index, every value; bit planes for the bit-wise path),
  * every worker is checked through properties that hold at any size: the message has exactly
    k_l - k_{l-1} entries, indices strictly ascending, values = g_i / p_l within 1e-6, and the band is a
    rank interval: fewer than k_l entries of the row are larger than its smallest member, at most k_{l-1}
    are larger than its largest one,
  * the dense mean is compared with the oracle's average of the emitted messages on every coordinate.
"""
import numpy as np
import pytest
import torch

from paper_2507_05508_b200 import workloads as wl

pytestmark = pytest.mark.gpu

VAL_RTOL = 1e-6
AGG_RTOL = 1e-6
MARGIN = 1e-9


@pytest.fixture(scope="module")
def B():
    from paper_2507_05508_b200 import binding
    binding.lib()
    return binding


def _topk_fullsize(B, ora, w, step, oracle_workers=(0,)):
    torch.cuda.set_device(0)
    k = wl.topk_schedule(w)
    L = len(k)
    p = None if w.adaptive else list(wl.geometric_probs(L))
    ctx = B.mlmc_create(0, w.d, w.M, 32)           # as bench.py's Runner does
    try:
        g = wl.gradients(w, step, "cuda")
        out = B.TopkBuffers(w.M, wl.max_band(k))
        dense = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
        B.mlmc_compress_topk(ctx, g, k, p, w.seed, step, out)
        B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, w.M, w.d, dense)
        assert B.mlmc_get_status(ctx) == B.MLMC_OK
        level, count, p_sel = out.level.tolist(), out.count.tolist(), out.p_sel.tolist()
        kk = [0] + list(k)
        msgs = []
        for m in range(w.M):
            l, n = level[m], count[m]
            assert 0 <= l < L and n == kk[l + 1] - kk[l]
            idx = out.idx[m, :n].to(torch.int64) & 0xFFFFFFFF
            val = out.val[m, :n]
            if n > 1:
                assert bool((idx[1:] > idx[:-1]).all())                  # strictly ascending, hence unique
            if n:
                assert int(idx[-1]) < w.d
                mag = g[m].float().abs()
                band = mag[idx]
                ref = (g[m].float()[idx].double() / p_sel[m])
                assert bool(((val.double() - ref).abs() <= VAL_RTOL * ref.abs()).all())
                lo, hi = band.min(), band.max()
                assert int((mag > lo).sum()) < kk[l + 1] <= int((mag >= lo).sum())
                assert int((mag > hi).sum()) <= kk[l] < int((mag >= hi).sum())
                del mag, band, ref
            msgs.append((out.idx[m, :n].cpu().numpy().view(np.uint32), out.val[m, :n].cpu().numpy()))
        if w.adaptive:
            # Every worker's probabilities and draw, recomputed with library sorts and fp64 sums (neither the CUDA
            # kernels nor the oracle): p_l = Delta_l / sum Delta from the sorted magnitudes (Lemma 3.4), and the level is
            # the one the worker's uniform selects, unless the uniform lies within the margin of a cdf boundary.
            us = B.mlmc_read_u(ctx, w.seed, step, w.M)
            edges = torch.tensor([0] + list(k), device="cuda")
            for m in range(w.M):
                mag2 = g[m].double().abs().sort(descending=True).values.square_()
                csum = torch.cat([torch.zeros(1, dtype=torch.float64, device="cuda"), mag2.cumsum(0)])
                delta = (csum[edges[1:]] - csum[edges[:-1]]).clamp_min(0).sqrt()
                pm = (delta / delta.sum()).cpu().numpy()
                cdf = np.cumsum(pm)
                assert abs(p_sel[m] - pm[level[m]]) <= 1e-9 * pm[level[m]]
                lo_c = cdf[level[m] - 1] if level[m] else 0.0
                assert lo_c - MARGIN <= us[m] < cdf[level[m]] + MARGIN or level[m] == L - 1
                del mag2, csum
        for m in oracle_workers:                                         # whole rows through the oracle
            row = wl.as_numpy_bits(g[m:m + 1])[0]
            o = ora.topk(row, k, p=p, seed=w.seed, step=step, worker=m)
            if o.margin < MARGIN and level[m] != o.level:
                o = ora.topk(row, k, p=p, seed=w.seed, step=step, worker=m, force_level=level[m])
            assert level[m] == o.level
            assert abs(p_sel[m] - o.p_sel) <= 1e-10 * o.p_sel
            assert np.array_equal(msgs[m][0], o.idx)
            assert np.all(np.abs(msgs[m][1].astype(np.float64) - o.val) <= VAL_RTOL * np.abs(o.val))
        ref, scale = ora.aggregate_topk(msgs, w.d)
        got = dense.cpu().numpy().astype(np.float64)
        assert not np.isnan(got).any()
        assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    finally:
        B.mlmc_destroy(ctx)


# Steps {0, last} of every config; the whole-row oracle comparison takes a worker or two per step (a 124M-entry row
# costs the oracle's full sort about half a minute), every other worker goes through the properties above.
@pytest.mark.parametrize("step,workers", [(0, (0, 15)), (wl.C3.steps - 1, (7,))])
def test_c3_full_size(B, ora, step, workers):
    _topk_fullsize(B, ora, wl.C3, step=step, oracle_workers=workers)


@pytest.mark.parametrize("step,workers", [(0, (0,)), (wl.C4.steps - 1, (31,))])
def test_c4_full_size(B, ora, step, workers):
    _topk_fullsize(B, ora, wl.C4, step=step, oracle_workers=workers)


@pytest.mark.parametrize("step,workers", [(0, (3,)), (wl.C5A.steps - 1, (6,))])
def test_c5a_full_size(B, ora, step, workers):
    _topk_fullsize(B, ora, wl.C5A, step=step, oracle_workers=workers)


@pytest.mark.parametrize("step,workers", [(0, (0, 5)), (wl.C5B.steps - 1, (2,))])
def test_c5b_full_size(B, ora, step, workers):
    w = wl.C5B
    torch.cuda.set_device(0)
    b = list(w.bits)
    widths = np.diff(np.concatenate([[0], b]))
    ctx = B.mlmc_create(0, w.d, w.M, 32)
    try:
        g = wl.gradients(w, step, "cuda")
        out = B.BitBuffers(w.M, w.d, int(widths.max()))
        dense = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
        B.mlmc_compress_bitwise(ctx, g, b, None, w.seed, step, out)
        B.mlmc_aggregate(ctx, B.MLMC_BITWISE, out, b, w.M, w.d, dense)
        assert B.mlmc_get_status(ctx) == B.MLMC_OK
        level, p_sel, gmax = out.level.tolist(), out.p_sel.tolist(), out.gmax.cpu().numpy()
        assert np.array_equal(gmax, g.abs().max(dim=1).values.cpu().numpy())       # the normaliser of every worker

        class Msg:
            pass

        msgs = []
        for m in range(w.M):
            mm = Msg()
            wv = int(widths[level[m]])
            mm.planes = out.planes[m, :1 + wv].cpu().numpy().view(np.uint32)
            mm.gmax, mm.level, mm.p_sel = float(gmax[m]), level[m], p_sel[m]
            msgs.append(mm)
        for m in workers:                                                  # whole rows through the oracle
            row = wl.as_numpy_bits(g[m:m + 1])[0]
            o = ora.bitwise(row, b, None, seed=w.seed, step=step, worker=m)
            if o.margin < MARGIN and level[m] != o.level:
                o = ora.bitwise(row, b, None, seed=w.seed, step=step, worker=m, force_level=level[m])
            assert level[m] == o.level and np.float32(o.gmax) == gmax[m]
            assert abs(p_sel[m] - o.p_sel) <= 1e-10 * o.p_sel
            assert np.array_equal(msgs[m].planes, o.planes)
        ref, scale = ora.aggregate_bitwise(msgs, b, w.d)
        got = dense.cpu().numpy().astype(np.float64)
        assert not np.isnan(got).any()
        assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    finally:
        B.mlmc_destroy(ctx)


# ----------------------------------------------------------------------------------------------
# the further compressors at the sizes bench.py times them (c3s, c5f, c5r)
# ----------------------------------------------------------------------------------------------
def test_c3s_full_size_stopk_many_segments(B, ora):
    """s-Top-k with L = 1000 segments and a given p on the c3 gradient: every worker's message is one segment of the
    sorted row (at most s entries); two whole rows go through the oracle, all go through the rank-interval property."""
    w = wl.C3S
    torch.cuda.set_device(0)
    s = w.seg_len
    L = -(-w.d // s)
    assert L == 1000
    p = list(wl.geometric_probs(L))
    ctx = B.mlmc_create(0, w.d, w.M, 32)
    try:
        for step in (0, w.steps - 1):
            g = wl.gradients(w, step, "cuda")
            out = B.TopkBuffers(w.M, s)
            dense = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
            B.mlmc_compress_stopk(ctx, g, s, p, w.seed, step, out)
            B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, w.M, w.d, dense)
            assert B.mlmc_get_status(ctx) == B.MLMC_OK
            level, count, p_sel = out.level.tolist(), out.count.tolist(), out.p_sel.tolist()
            msgs = []
            for m in range(w.M):
                l, n = level[m], count[m]
                lo, hi = s * l, min(w.d, s * (l + 1))
                assert 0 <= l < L and n == hi - lo
                idx = out.idx[m, :n].to(torch.int64) & 0xFFFFFFFF
                assert bool((idx[1:] > idx[:-1]).all()) and int(idx[-1]) < w.d
                mag = g[m].abs()
                band = mag[idx]
                assert int((mag > band.min()).sum()) < hi <= int((mag >= band.min()).sum())
                assert int((mag > band.max()).sum()) <= lo < int((mag >= band.max()).sum())
                ref = g[m][idx].double() / p_sel[m]
                assert bool(((out.val[m, :n].double() - ref).abs() <= VAL_RTOL * ref.abs()).all())
                msgs.append((out.idx[m, :n].cpu().numpy().view(np.uint32), out.val[m, :n].cpu().numpy()))
            for m in (1, w.M - 1):
                o = ora.stopk(wl.as_numpy_bits(g[m:m + 1])[0], s, p, seed=w.seed, step=step, worker=m)
                if o.margin < MARGIN and level[m] != o.level:
                    o = ora.stopk(wl.as_numpy_bits(g[m:m + 1])[0], s, p, seed=w.seed, step=step, worker=m, force_level=level[m])
                assert level[m] == o.level and abs(p_sel[m] - o.p_sel) <= 1e-12 * o.p_sel
                assert np.array_equal(msgs[m][0], o.idx)
            ref, scale = ora.aggregate_topk(msgs, w.d)
            got = dense.cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    finally:
        B.mlmc_destroy(ctx)


def test_c3a_full_size_stopk_adaptive_many_segments(B, ora):
    """s-Top-k with L = 100 segments and adaptive p (Lemma 3.4) on the c3 gradient, the sorted path at the size
    bench.py times it (the 16 rows are sorted in two groups).  Every worker: the band is the rank interval of its
    segment, and p_sel and the draw agree with segment norms recomputed by library sorts and fp64 sums; two whole rows
    go through the oracle."""
    w = wl.C3A
    torch.cuda.set_device(0)
    s = w.seg_len
    L = -(-w.d // s)
    assert L == 100 and w.adaptive
    ctx = B.mlmc_create(0, w.d, w.M, 32)
    try:
        for step in (0, w.steps - 1):
            g = wl.gradients(w, step, "cuda")
            out = B.TopkBuffers(w.M, s)
            dense = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
            B.mlmc_compress_stopk(ctx, g, s, None, w.seed, step, out)
            B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, w.M, w.d, dense)
            assert B.mlmc_get_status(ctx) == B.MLMC_OK
            level, count, p_sel = out.level.tolist(), out.count.tolist(), out.p_sel.tolist()
            us = B.mlmc_read_u(ctx, w.seed, step, w.M)
            edges = torch.arange(0, L + 1, device="cuda").mul_(s).clamp_(max=w.d)
            msgs = []
            for m in range(w.M):
                l, n = level[m], count[m]
                lo, hi = s * l, min(w.d, s * (l + 1))
                assert 0 <= l < L and n == hi - lo
                idx = out.idx[m, :n].to(torch.int64) & 0xFFFFFFFF
                assert bool((idx[1:] > idx[:-1]).all()) and int(idx[-1]) < w.d
                mag = g[m].abs()
                band = mag[idx]
                assert int((mag > band.min()).sum()) < hi <= int((mag >= band.min()).sum())
                assert int((mag > band.max()).sum()) <= lo < int((mag >= band.max()).sum())
                mag2 = mag.double().sort(descending=True).values.square_()
                csum = torch.cat([torch.zeros(1, dtype=torch.float64, device="cuda"), mag2.cumsum(0)])
                delta = (csum[edges[1:]] - csum[edges[:-1]]).clamp_min(0).sqrt()
                pm = (delta / delta.sum()).cpu().numpy()
                cdf = np.cumsum(pm)
                assert abs(p_sel[m] - pm[l]) <= 1e-9 * pm[l]
                assert ((cdf[l - 1] if l else 0.0) - MARGIN <= us[m] < cdf[l] + MARGIN) or l == L - 1
                ref = g[m][idx].double() / p_sel[m]
                assert bool(((out.val[m, :n].double() - ref).abs() <= VAL_RTOL * ref.abs()).all())
                msgs.append((out.idx[m, :n].cpu().numpy().view(np.uint32), out.val[m, :n].cpu().numpy()))
            for m in (0, w.M - 1):                                       # one row of each group
                o = ora.stopk(wl.as_numpy_bits(g[m:m + 1])[0], s, None, seed=w.seed, step=step, worker=m)
                if o.margin < MARGIN and level[m] != o.level:
                    o = ora.stopk(wl.as_numpy_bits(g[m:m + 1])[0], s, None, seed=w.seed, step=step, worker=m, force_level=level[m])
                assert level[m] == o.level and abs(p_sel[m] - o.p_sel) <= 1e-11 * o.p_sel
                assert np.array_equal(msgs[m][0], o.idx)
            ref, scale = ora.aggregate_topk(msgs, w.d)
            got = dense.cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    finally:
        B.mlmc_destroy(ctx)


def test_c5f_full_size_floatbits(B, ora):
    """Floating-point MLMC on the c5 gradient.  The compressor is element-wise and its probabilities are fixed, so the
    oracle on a prefix of a row gives that prefix of the message: the first 2^22 coordinates of every worker (exponent
    bytes, planes, dense mean), and the last, ragged plane words of the row."""
    w = wl.C5F
    torch.cuda.set_device(0)
    mb = list(w.bits)
    widths = np.diff(np.concatenate([[0], mb]))
    n_pre = 1 << 22
    ctx = B.mlmc_create(0, w.d, w.M, 32)
    try:
        for step in (0, w.steps - 1):
            g = wl.gradients(w, step, "cuda")
            out = B.FloatBuffers(w.M, w.d, int(widths.max()))
            dense = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
            B.mlmc_compress_floatbits(ctx, g, mb, None, w.seed, step, out)
            B.mlmc_aggregate_floatbits(ctx, out, mb, w.M, w.d, dense)
            assert B.mlmc_get_status(ctx) == B.MLMC_OK
            level = out.level.tolist()
            rows = []
            tail0 = (w.d - 4096) // 32 * 32                     # a word-aligned tail that ends at d
            for m in range(w.M):
                wv = int(widths[level[m]])
                for lo, hi in ((0, n_pre), (tail0, w.d)):
                    o = ora.floatbits(g[m, lo:hi].cpu().numpy(), mb, None, seed=w.seed, step=step, worker=m,
                                      force_level=level[m])
                    assert np.array_equal(out.expo[m, lo:hi].cpu().numpy(), o.expo)
                    got_planes = out.planes[m, :1 + wv, lo // 32:(hi + 31) // 32].cpu().numpy().view(np.uint32)
                    assert np.array_equal(got_planes, o.planes)
                    if lo == 0:
                        rows.append(o.est)
                full = ora.floatbits(g[m, :1024].cpu().numpy(), mb, None, seed=w.seed, step=step, worker=m)
                assert full.margin < MARGIN or full.level == level[m]      # the draw does not depend on the data
                assert abs(float(out.p_sel[m]) - full.p[level[m]]) <= 1e-15
            ref, scale = ora.aggregate_dense(rows, n_pre)
            got = dense[:n_pre].cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
            assert bool(torch.isfinite(dense).all())
    finally:
        B.mlmc_destroy(ctx)


def test_c5r_full_size_rtn(B, ora):
    """Adaptive MLMC-RTN on the c5 gradient: whole rows through the oracle (no sort: a few seconds per row) for two
    workers, the clipping value of every worker, and the dense mean against the oracle's average of the emitted dense
    messages on a slice of the coordinates."""
    w = wl.C5R
    torch.cuda.set_device(0)
    r = list(w.bits)
    ctx = B.mlmc_create(0, w.d, w.M, 32)
    try:
        for step, workers in ((0, (0, 5)), (w.steps - 1, (7,))):
            g = wl.gradients(w, step, "cuda")
            out = B.RtnBuffers(w.M, w.d)
            dense = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
            B.mlmc_compress_rtn(ctx, g, r, None, w.seed, step, out)
            B.mlmc_aggregate_rtn(ctx, out, w.M, w.d, dense)
            assert B.mlmc_get_status(ctx) == B.MLMC_OK
            level, p_sel, c = out.level.tolist(), out.p_sel.tolist(), out.c.cpu().numpy()
            assert np.array_equal(c, g.abs().max(dim=1).values.cpu().numpy())
            for m in workers:
                row = wl.as_numpy_bits(g[m:m + 1])[0]
                o = ora.rtn(row, r, None, seed=w.seed, step=step, worker=m)
                if o.margin < MARGIN and level[m] != o.level:
                    o = ora.rtn(row, r, None, seed=w.seed, step=step, worker=m, force_level=level[m])
                assert level[m] == o.level and abs(p_sel[m] - o.p_sel) <= 1e-10 * o.p_sel
                got = out.val[m, :w.d].cpu().numpy().astype(np.float64)
                assert np.all(np.abs(got - o.val) <= VAL_RTOL * np.abs(o.val) + 1e-45)
                del got, o, row
            lo, hi = 40_000_000, 40_000_000 + (1 << 22)
            rows = [out.val[m, lo:hi].cpu().numpy() for m in range(w.M)]
            ref, scale = ora.aggregate_dense(rows, hi - lo)
            got = dense[lo:hi].cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
            assert bool(torch.isfinite(dense).all())
    finally:
        B.mlmc_destroy(ctx)
