"""GPU parity of the further multilevel compressors (s-Top-k, floating-point bit-wise, RTN), called through the
C ABI, against the CPU oracle on the same seeded inputs.

Bar as for the other parity tests: sampled levels bit-exact (draws within 1e-9 of a cdf boundary excluded and
counted), indices, exponent bytes and bit planes bit-exact, message values within 1e-6 relative, aggregated means
within 1e-6 (1/M) sum_m |term_m| per coordinate.
"""
import math

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


@pytest.fixture(scope="module")
def ctx(B):
    c = B.mlmc_create(0, 1_100_000, 16, 32)
    yield c
    B.mlmc_destroy(c)


def padded(g: torch.Tensor, mult: int) -> torch.Tensor:
    M, d = g.shape
    ld = (d + mult - 1) // mult * mult
    buf = torch.zeros((M, ld), dtype=g.dtype, device=g.device)
    buf[:, :d] = g
    return buf[:, :d]


def to_dev(g_np: np.ndarray) -> torch.Tensor:
    return padded(torch.from_numpy(np.ascontiguousarray(g_np)).cuda(), 4)


# ----------------------------------------------------------------------------------------------
# floating-point bit-wise MLMC (App. B)
# ----------------------------------------------------------------------------------------------
def check_floatbits(B, ora, ctx, g, mb, p, seed, step):
    M, d = g.shape
    widths = np.diff(np.concatenate([[0], mb]))
    out = B.FloatBuffers(M, d, int(widths.max()))
    dense = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    B.mlmc_compress_floatbits(ctx, g, mb, p, seed, step, out)
    B.mlmc_aggregate_floatbits(ctx, out, mb, M, d, dense)
    assert B.mlmc_get_status(ctx) == B.MLMC_OK
    gh = wl.as_numpy_bits(g)
    level, p_sel = out.level.cpu().numpy(), out.p_sel.cpu().numpy()
    expo = out.expo.cpu().numpy()
    planes = out.planes.cpu().numpy().view(np.uint32)
    rows = []
    for m in range(M):
        o = ora.floatbits(gh[m], mb, p, seed=seed, step=step, worker=m)
        if o.margin < MARGIN and level[m] != o.level:
            o = ora.floatbits(gh[m], mb, p, seed=seed, step=step, worker=m, force_level=int(level[m]))
        assert level[m] == o.level
        assert abs(p_sel[m] - o.p_sel) <= 1e-15
        assert np.array_equal(expo[m, :d], o.expo), f"worker {m}: exponent bytes differ"
        assert not expo[m, d:].any()
        w = int(widths[o.level])
        assert np.array_equal(planes[m, :1 + w], o.planes), f"worker {m}: planes differ"
        rows.append(o.est)
    ref, scale = ora.aggregate_dense(rows, d)
    got = dense.cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_floatbits_parity(B, ora, ctx, dtype):
    w = wl.shrink(wl.C5B, 333_337, 5)
    sc = wl.scales(w, "cuda")
    top = 23 if dtype == "f32" else 7
    schedules = ([1, 2, 4, 8, 16, 23], list(range(1, 24)), [23]) if dtype == "f32" else ([1, 3, 7], list(range(1, 8)))
    for step in range(3):
        g = wl.gradients(w, step, "cuda", sc)
        g = padded(g.to(torch.bfloat16), 8) if dtype == "bf16" else padded(g, 4)
        for mb in schedules:
            assert mb[-1] == top
            check_floatbits(B, ora, ctx, g, mb, None, w.seed, step)            # App. B's optimal fixed probabilities
        L = len(schedules[0])
        check_floatbits(B, ora, ctx, g, schedules[0], [1.0 / L] * L, w.seed, step + 10)


def test_floatbits_degenerate_and_errors(B, ora, ctx):
    z = to_dev(np.zeros((2, 1000), dtype=np.float32))
    check_floatbits(B, ora, ctx, z, [1, 23], None, 0, 0)
    rng = np.random.default_rng(51)
    odd = rng.choice(np.array([0.0, -0.0, 1e-45, -3e-41, 1.17549435e-38, -1.5, 3e30], dtype=np.float32), (3, 4099))
    for step in range(4):
        check_floatbits(B, ora, ctx, to_dev(odd), [2, 9, 23], [0.5, 0.25, 0.25], 1, step)
    g = to_dev(rng.standard_normal((2, 5000)).astype(np.float32))
    out = B.FloatBuffers(2, 5000, 8)
    bad = g.clone()
    bad[1, 4321] = float("inf")
    B.mlmc_compress_floatbits(ctx, bad, list(range(1, 24)), None, 0, 0, out)
    assert B.mlmc_get_status(ctx) == B.MLMC_ERR_NONFINITE
    assert out.level.tolist()[1] == -1 and out.level.tolist()[0] >= 0
    dense = torch.zeros(5000, device="cuda")
    B.mlmc_aggregate_floatbits(ctx, out, list(range(1, 24)), 2, 5000, dense)     # the void message adds nothing
    assert torch.isfinite(dense).all()
    for mb, code in (([1, 2, 22], B.MLMC_ERR_SCHEDULE), ([2, 2, 23], B.MLMC_ERR_SCHEDULE), ([1, 24], B.MLMC_ERR_SCHEDULE)):
        with pytest.raises(B.MlmcError) as e:
            B.mlmc_compress_floatbits(ctx, g, mb, None, 0, 0, out)
        assert e.value.code == code
    small = B.FloatBuffers(2, 5000, 2)                                            # too few planes for a 7-digit field
    B.mlmc_compress_floatbits(ctx, g, [16, 23], [0.01, 0.99], 0, 0, small)
    assert B.mlmc_get_status(ctx) == B.MLMC_ERR_CAPACITY


# ----------------------------------------------------------------------------------------------
# MLMC-RTN (App. G)
# ----------------------------------------------------------------------------------------------
def check_rtn(B, ora, ctx, g, r, p, seed, step, expect_excluded=1):
    M, d = g.shape
    out = B.RtnBuffers(M, d)
    dense = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    B.mlmc_compress_rtn(ctx, g, r, p, seed, step, out)
    B.mlmc_aggregate_rtn(ctx, out, M, d, dense)
    assert B.mlmc_get_status(ctx) == B.MLMC_OK
    gh = wl.as_numpy_bits(g)
    level, p_sel, c = out.level.cpu().numpy(), out.p_sel.cpu().numpy(), out.c.cpu().numpy()
    val = out.val.cpu().numpy()[:, :d]
    excluded, rows = 0, []
    for m in range(M):
        o = ora.rtn(gh[m], r, p, seed=seed, step=step, worker=m)
        if o.margin < MARGIN and level[m] != o.level:
            excluded += 1
            o = ora.rtn(gh[m], r, p, seed=seed, step=step, worker=m, force_level=int(level[m]))
        assert level[m] == o.level, f"worker {m}: level {level[m]} vs {o.level} (margin {o.margin})"
        assert c[m] == np.float32(o.c)
        assert abs(p_sel[m] - o.p_sel) <= 1e-11 * max(o.p_sel, 1e-300) + 1e-15
        assert np.all(np.abs(val[m].astype(np.float64) - o.val) <= VAL_RTOL * np.abs(o.val) + 1e-45)
        rows.append(o.val)
    ref, scale = ora.aggregate_dense(rows, d)
    got = dense.cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    assert excluded <= expect_excluded


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rtn_parity(B, ora, ctx, dtype):
    w = wl.shrink(wl.C5A, 250_003, 4)
    sc = wl.scales(w, "cuda")
    for step in range(3):
        g = wl.gradients(w, step, "cuda", sc)
        g = padded(g.to(torch.bfloat16), 8) if dtype == "bf16" else padded(g, 4)
        check_rtn(B, ora, ctx, g, [2, 4, 8, 16], None, w.seed, step)             # the paper's widths, adaptive (Alg. 3)
        check_rtn(B, ora, ctx, g, [2, 4, 8, 16], [0.3, 0.3, 0.2, 0.1, 0.1], w.seed, step)
        check_rtn(B, ora, ctx, g, list(range(1, 17)), None, w.seed, step, expect_excluded=2)   # 17 levels
        check_rtn(B, ora, ctx, g, [], None, w.seed, step)                         # the identity alone


def test_rtn_level_probs_and_degenerate(B, ora, ctx):
    rng = np.random.default_rng(52)
    g_np = (rng.standard_normal((3, 70_001)) * 10.0 ** rng.uniform(-2, 0, (3, 1))).astype(np.float32)
    g = to_dev(g_np)
    r = [2, 4, 8, 16]
    p_out = torch.zeros((3, 5), dtype=torch.float64, device="cuda")
    d_out = torch.zeros((3, 5), dtype=torch.float64, device="cuda")
    B.mlmc_level_probs(ctx, g, B.MLMC_RTN, r, None, p_out, d_out)
    assert B.mlmc_get_status(ctx) == 0
    for m in range(3):
        o = ora.rtn(g_np[m], r, None)
        assert np.allclose(p_out[m].cpu().numpy(), o.p, rtol=1e-11, atol=1e-15)
        assert np.allclose(d_out[m].cpu().numpy(), o.delta, rtol=1e-12, atol=0)
    check_rtn(B, ora, ctx, to_dev(np.zeros((2, 999), dtype=np.float32)), r, None, 0, 0)
    one = np.zeros((2, 1000), dtype=np.float32)
    one[0, 17], one[1, 999] = -1e-40, 5.0
    check_rtn(B, ora, ctx, to_dev(one), r, None, 0, 1)
    with pytest.raises(B.MlmcError) as e:
        B.mlmc_compress_rtn(ctx, g, [4, 2], None, 0, 0, B.RtnBuffers(3, 70_001))
    assert e.value.code == B.MLMC_ERR_SCHEDULE
    bad = padded(g.clone(), 4)
    bad[2, 5] = float("nan")
    out = B.RtnBuffers(3, 70_001)
    B.mlmc_compress_rtn(ctx, bad, r, None, 0, 0, out)
    assert B.mlmc_get_status(ctx) == B.MLMC_ERR_NONFINITE and out.level.tolist()[2] == -1


# ----------------------------------------------------------------------------------------------
# s-Top-k (Sec. 2.2, App. D)
# ----------------------------------------------------------------------------------------------
def check_stopk(B, ora, ctx, g, s, p, seed, step, expect_excluded=1):
    M, d = g.shape
    out = B.TopkBuffers(M, min(s, d))
    dense = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    B.mlmc_compress_stopk(ctx, g, s, p, seed, step, out)
    B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, M, d, dense)
    assert B.mlmc_get_status(ctx) == B.MLMC_OK
    gh = wl.as_numpy_bits(g)
    level, count, p_sel = out.level.cpu().numpy(), out.count.cpu().numpy(), out.p_sel.cpu().numpy()
    idx_all, val_all = out.idx.cpu().numpy().view(np.uint32), out.val.cpu().numpy()
    excluded, msgs = 0, []
    for m in range(M):
        o = ora.stopk(gh[m], s, p, seed=seed, step=step, worker=m)
        if o.margin < MARGIN and level[m] != o.level:
            excluded += 1
            o = ora.stopk(gh[m], s, p, seed=seed, step=step, worker=m, force_level=int(level[m]))
        assert level[m] == o.level
        assert abs(p_sel[m] - o.p_sel) <= 1e-11 * max(o.p_sel, 1e-300) + 1e-15
        n = int(count[m])
        assert n == o.idx.size and np.array_equal(idx_all[m, :n], o.idx)
        assert np.all(np.abs(val_all[m, :n].astype(np.float64) - o.val) <= VAL_RTOL * np.abs(o.val))
        msgs.append((o.idx, o.val))
    ref, scale = ora.aggregate_topk(msgs, d)
    got = dense.cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    assert excluded <= expect_excluded


def test_stopk_few_segments_adaptive_and_fixed(B, ora, ctx):
    w = wl.shrink(wl.C3, 200_003, 4)
    sc = wl.scales(w, "cuda")
    for step in range(3):
        g = padded(wl.gradients(w, step, "cuda", sc), 4)
        check_stopk(B, ora, ctx, g, 10_000, None, w.seed, step)                   # L = 21 segments, Lemma 3.4
        L = 21
        check_stopk(B, ora, ctx, g, 10_000, list(wl.geometric_probs(L)), w.seed, step)
        check_stopk(B, ora, ctx, g, 200_003, None, w.seed, step)                  # one segment: the identity


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stopk_many_segments_fixed_p(B, ora, ctx, dtype):
    """L = ceil(d / s) far beyond MLMC_MAX_LEVELS: the uniform-segment regime of Sec. 2.2 / Lemma 3.6 with a given p."""
    rng = np.random.default_rng(53)
    d, s = 150_001, 500
    L = -(-d // s)
    assert L == 301
    g_np = (rng.standard_normal((3, d)) * 10.0 ** rng.uniform(-3, 0, (3, d))).astype(np.float32)
    g_np[:, ::7] = np.round(g_np[:, ::7], 3)                                       # ties across segment boundaries
    g = to_dev(g_np)
    if dtype == "bf16":
        g = padded(g.to(torch.bfloat16), 8)
    harmonic = 1.0 / np.arange(1, L + 1)
    for step, p in enumerate(([1.0 / L] * L, list(harmonic / harmonic.sum()), [1.0 / L] * L, [1.0 / L] * L)):
        check_stopk(B, ora, ctx, g, s, p, 17, step, expect_excluded=0)
    # the last, shorter segment (level L - 1) and the first one
    for l in (0, L - 1, L - 2):
        p = np.full(L, 1e-9)
        p[l] = 1.0 - 1e-9 * (L - 1)
        check_stopk(B, ora, ctx, g, s, list(p), 3, l, expect_excluded=0)
    out = B.TopkBuffers(3, s)
    with pytest.raises(B.MlmcError) as e:
        B.mlmc_compress_stopk(ctx, g, s, [1.0 / L] * (L - 1) + [0.0], 0, 0, out)
    assert e.value.code == B.MLMC_ERR_PROB


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stopk_many_segments_adaptive(B, ora, ctx, dtype):
    """Adaptive p (Lemma 3.4: p^l proportional to the norm of segment l) with L = 101 and L = 33 segments, the regime of
    the paper's Adaptive MLMC-Top-k runs (segments of 1 % of the vector and more): every segment norm comes from a
    sort of the row's magnitude keys."""
    rng = np.random.default_rng(55)
    d = 150_001
    g_np = (rng.standard_normal((3, d)) * 10.0 ** rng.uniform(-3, 0, (3, d))).astype(np.float32)
    g_np[:, ::7] = np.round(g_np[:, ::7], 3)                                       # ties across segment boundaries
    g_np[2, 1000:] = 0.0                                                           # a row that is mostly zero: empty tail segments
    g = to_dev(g_np)
    if dtype == "bf16":
        g = padded(g.to(torch.bfloat16), 8)
    for s, steps in ((1500, 6), (4600, 3)):
        assert -(-d // s) in (101, 33)
        for step in range(steps):
            check_stopk(B, ora, ctx, g, s, None, 23, step, expect_excluded=1)
    z = to_dev(np.zeros((2, 5000), dtype=np.float32))
    check_stopk(B, ora, ctx, z, 50, None, 1, 0)                                    # all zero: level 0 with p = 1
    small = to_dev(rng.standard_normal((2, 70)).astype(np.float32))
    check_stopk(B, ora, ctx, small, 1, None, 1, 1)                                 # s = 1: Top-k with the unit schedule, L = 70


@pytest.mark.parametrize("d,s", [(8192, 100), (8193, 100), (16384, 37), (131_077, 1), (40_000, 1023), (40_000, 1024), (200_000, 4096), (200_000, 4097)])
def test_stopk_adaptive_sort_edges(B, ora, ctx, d, s):
    """The sorted path at the edges of its tiling: rows of exactly one and two sort tiles and one key more, one
    entry per segment (L = d), and segment lengths on both sides of the switch between a warp and a block per
    segment and of the chunk length of the norms."""
    rng = np.random.default_rng(59 + d + s)
    g_np = (rng.standard_normal((2, d)) * 10.0 ** rng.uniform(-2, 0, (2, d))).astype(np.float32)
    g_np[:, ::5] = np.round(g_np[:, ::5], 2)                                       # ties
    g = to_dev(g_np)
    assert -(-d // s) > 32
    for step in range(2):
        check_stopk(B, ora, ctx, g, s, None, 31, step, expect_excluded=1)


def test_stopk_adaptive_rows_sorted_in_groups(B, ora):
    """A context whose rows are too long to be sorted all together (the scratch memory of the sort holds two of its
    three rows): the second group reuses the buffers of the first."""
    rng = np.random.default_rng(57)
    d = 60_011
    g = to_dev((rng.standard_normal((3, d)) * 10.0 ** rng.uniform(-3, 0, (3, d))).astype(np.float32))
    big = B.mlmc_create(0, 48_000_000, 3, 32)
    try:
        for step in range(3):
            check_stopk(B, ora, big, g, 601, None, 29, step, expect_excluded=1)   # L = 100
    finally:
        B.mlmc_destroy(big)


def test_stopk_exponential_decay_closed_forms(B, ora, ctx):
    """Assumption 3.5 / Lemma 3.6 on the device: |v(j)| = a exp(-r j / 2) on the sorted vector, s L = d with L = 32
    segments; the residual norms of mlmc_level_probs follow the closed form of App. E, and the adaptive second moment
    (sum Delta)^2 - ||v||^2 is the lemma's variance."""
    rng = np.random.default_rng(54)
    d, s, r, a = 32_768, 1024, 0.0005, 3.0
    L = d // s
    mags = a * np.exp(-0.5 * r * np.arange(d))
    g_np = np.empty((2, d), dtype=np.float32)
    for m in range(2):
        pi = rng.permutation(d)
        g_np[m, pi] = (mags * rng.choice([-1.0, 1.0], d)).astype(np.float32)
    g = to_dev(g_np)
    k = [s * (l + 1) for l in range(L)]
    p_out = torch.zeros((2, L), dtype=torch.float64, device="cuda")
    d_out = torch.zeros((2, L), dtype=torch.float64, device="cuda")
    B.mlmc_level_probs(ctx, g, B.MLMC_TOPK, k, None, p_out, d_out)
    assert B.mlmc_get_status(ctx) == 0
    lvl = np.arange(1, L + 1)
    delta2 = a ** 2 * np.exp(-r * s * (lvl - 1)) * (1 - math.exp(-r * s)) / (1 - math.exp(-r))
    norm2 = a ** 2 * (1 - math.exp(-r * d)) / (1 - math.exp(-r))
    exact_var = norm2 * ((1 - math.exp(-r * s)) / (1 - math.exp(-r * d))
                         * ((1 - math.exp(-0.5 * r * d)) / (1 - math.exp(-0.5 * r * s))) ** 2 - 1)
    for m in range(2):
        dl = d_out[m].cpu().numpy()
        assert np.allclose(dl ** 2, delta2, rtol=2e-6)
        assert np.allclose(p_out[m].cpu().numpy(), np.sqrt(delta2) / np.sqrt(delta2).sum(), rtol=2e-6)
        assert dl.sum() ** 2 - float(np.sum(g_np[m].astype(np.float64) ** 2)) == pytest.approx(exact_var, rel=1e-4)
    check_stopk(B, ora, ctx, g, s, None, 2, 0)
