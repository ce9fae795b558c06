"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Bar: bit-exact sampled levels (draws whose uniform lies within 1e-9 of a cdf boundary are excluded and
counted) and band indices; message values within 1e-6 relative; aggregated means within
1e-6 * (1/M) sum_m |term_m| per coordinate (the conditioning scale of the fp32 sum).
"""
import math
import os

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
    c = B.mlmc_create(0, 2_200_000, 32, 32)
    yield c
    B.mlmc_destroy(c)


def padded(g: torch.Tensor, mult: int) -> torch.Tensor:
    """Copy [M, d] into a buffer whose row stride is a multiple of `mult` elements (16-byte rows)."""
    M, d = g.shape
    ld = (d + mult - 1) // mult * mult
    buf = torch.zeros((M, ld), dtype=g.dtype, device=g.device)
    buf[:, :d] = g
    return buf[:, :d]


def to_dev(g_np: np.ndarray) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(g_np)).cuda()
    return padded(t, 4)


def check_topk(B, ora, ctx, g: torch.Tensor, k, p, seed, step, capacity=None, expect_excluded=0):
    """Runs compress + aggregate on the GPU and compares every worker with the oracle. Returns #excluded draws."""
    M, d = g.shape
    cap = capacity if capacity is not None else wl.max_band(k)
    out = B.TopkBuffers(M, cap)
    dense = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    B.mlmc_compress_topk(ctx, g, k, p, seed, step, out)
    B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, M, d, dense)
    assert B.mlmc_get_status(ctx) == B.MLMC_OK
    g_host = wl.as_numpy_bits(g)
    level, count, p_sel = out.level.cpu().numpy(), out.count.cpu().numpy(), out.p_sel.cpu().numpy()
    idx_all = out.idx.cpu().numpy().view(np.uint32)
    val_all = out.val.cpu().numpy()
    excluded = 0
    msgs = []
    for m in range(M):
        o = ora.topk(g_host[m], k, p=p, seed=seed, step=step, worker=m)
        if o.margin < MARGIN and level[m] != o.level:
            excluded += 1
            o = ora.topk(g_host[m], k, p=p, seed=seed, step=step, worker=m, force_level=int(level[m]))
        assert level[m] == o.level, f"worker {m}: level {level[m]} vs oracle {o.level} (margin {o.margin})"
        assert abs(p_sel[m] - o.p_sel) <= 1e-11 * max(o.p_sel, 1e-300) + 1e-15
        n = int(count[m])
        assert n == o.idx.size
        assert np.array_equal(idx_all[m, :n], o.idx), f"worker {m}: band indices differ"
        assert np.all(np.abs(val_all[m, :n].astype(np.float64) - o.val) <= VAL_RTOL * np.abs(o.val))
        msgs.append((o.idx, o.val))
    ref, scale = ora.aggregate_topk(msgs, d)
    got = dense.cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()                      # every element written
    assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    assert excluded <= expect_excluded
    return excluded


def check_bitwise(B, ora, ctx, g: torch.Tensor, b, p, seed, step):
    M, d = g.shape
    widths = np.diff(np.concatenate([[0], b]))
    out = B.BitBuffers(M, d, int(widths.max()))
    dense = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    B.mlmc_compress_bitwise(ctx, g, b, p, seed, step, out)
    B.mlmc_aggregate(ctx, B.MLMC_BITWISE, out, b, M, d, dense)
    assert B.mlmc_get_status(ctx) == B.MLMC_OK
    g_host = wl.as_numpy_bits(g)
    level, p_sel, gmax = out.level.cpu().numpy(), out.p_sel.cpu().numpy(), out.gmax.cpu().numpy()
    planes = out.planes.cpu().numpy().view(np.uint32)
    excluded = 0
    msgs = []
    for m in range(M):
        o = ora.bitwise(g_host[m], b, p=p, seed=seed, step=step, worker=m)
        if o.margin < MARGIN and level[m] != o.level:
            excluded += 1
            o = ora.bitwise(g_host[m], b, p=p, seed=seed, step=step, worker=m, force_level=int(level[m]))
        assert level[m] == o.level
        assert gmax[m] == np.float32(o.gmax)
        assert abs(p_sel[m] - o.p_sel) <= 1e-11 * max(o.p_sel, 1e-300) + 1e-15
        w = int(widths[o.level])
        assert np.array_equal(planes[m, :1 + w], o.planes), f"worker {m}: bit planes differ"
        msgs.append(o)
    ref, scale = ora.aggregate_bitwise(msgs, b, d)
    got = dense.cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    assert np.all(np.abs(got - ref) <= AGG_RTOL * scale + 1e-45)
    return excluded


# ----------------------------------------------------------------------------------------------
def test_counter_rng_matches_known_answers(B, ora, ctx):
    path = os.path.join(os.path.dirname(__file__), "golden", "rng_kat.txt")
    for ln in open(path):
        if ln.startswith("#"):
            continue
        s, t, w, _, u = ln.split()
        s, t, w = int(s), int(t), int(w)
        if w < 32:
            assert B.mlmc_read_u(ctx, s, t, w + 1)[w] == float.fromhex(u)
    u = B.mlmc_read_u(ctx, 77, 123456789, 32)
    assert u == [ora.uniform(77, 123456789, m) for m in range(32)]


def test_c1_all_steps(B, ora, ctx):
    w = wl.C1
    k, p = wl.topk_schedule(w), wl.geometric_probs(11)
    assert len(k) == 11 and k[-1] == w.d
    sc = wl.scales(w, "cuda")
    excluded = 0
    for step in range(w.steps):
        g = wl.gradients(w, step, "cuda", sc)
        excluded += check_topk(B, ora, ctx, g, k, list(p), w.seed, step, expect_excluded=1)
    assert excluded <= 1


def test_c1_adaptive(B, ora, ctx):
    w = wl.C1
    k = wl.topk_schedule(w)
    g = wl.gradients(w, 3, "cuda")
    for step in range(4):
        check_topk(B, ora, ctx, g, k, None, 5, step, expect_excluded=1)


@pytest.mark.parametrize("name,d,M", [("c3", 300_007, 5), ("c5a", 700_001, 3)])
def test_topk_fp32_segments(B, ora, ctx, name, d, M):
    base = wl.ALL[name]
    w = wl.shrink(base, d, M)
    k = wl.topk_schedule(w)
    p = None if w.adaptive else list(wl.geometric_probs(len(k)))
    sc = wl.scales(w, "cuda")
    for step in (0, 1, 7):
        g = padded(wl.gradients(w, step, "cuda", sc), 4)
        check_topk(B, ora, ctx, g, k, p, w.seed, step, expect_excluded=1)


def test_topk_bf16_adaptive(B, ora, ctx):
    w = wl.shrink(wl.C4, 400_003, 6)
    k = wl.topk_schedule(w)
    sc = wl.scales(w, "cuda")
    for step in (0, 5):
        g = padded(wl.gradients(w, step, "cuda", sc), 8)
        check_topk(B, ora, ctx, g, k, None, w.seed, step, expect_excluded=1)
        check_topk(B, ora, ctx, g, k, list(wl.geometric_probs(len(k))), w.seed, step, expect_excluded=1)


def test_topk_every_level_is_reachable(B, ora, ctx):
    # force each level in turn with a near-one-hot fixed p: all bands, both thresholds, are exercised
    rng = np.random.default_rng(21)
    d = 50_001
    g_np = (rng.standard_normal((2, d)) * 10.0 ** rng.uniform(-3, 0, (2, d))).astype(np.float32)
    g_np[:, ::5] = np.round(g_np[:, ::5], 2)             # ties
    g = to_dev(g_np)
    k = [1, 2, 50, 50, 1000, 1001, 25_000, 50_000, d]
    for l in range(len(k)):
        p = np.full(len(k), 1e-6)
        p[l] = 1.0 - 1e-6 * (len(k) - 1)
        check_topk(B, ora, ctx, g, k, list(p), 1, l, expect_excluded=0)


@pytest.mark.parametrize("case", ["all_equal", "all_zero", "ties", "outlier", "signed_zero_denormal", "tiny_d"])
def test_topk_degenerate_inputs(B, ora, ctx, case):
    rng = np.random.default_rng(22)
    d = 10_003
    if case == "all_equal":
        g_np = np.full((2, d), -0.75, dtype=np.float32)
    elif case == "all_zero":
        g_np = np.zeros((2, d), dtype=np.float32)
    elif case == "ties":
        g_np = rng.integers(-4, 5, (2, d)).astype(np.float32)
    elif case == "outlier":
        g_np = rng.standard_normal((2, d)).astype(np.float32) * 1e-6
        g_np[0, 777] = 3e30
        g_np[1, d - 1] = -3e30
    elif case == "signed_zero_denormal":
        g_np = rng.choice(np.array([0.0, -0.0, 1e-45, -1e-45, 1e-39, 1.0], dtype=np.float32), (2, d))
    else:
        d = 5
        g_np = rng.standard_normal((1, d)).astype(np.float32)
    g = to_dev(g_np)
    k = [1, 3, 5] if d == 5 else [1, 10, 100, 100, 5000, d]
    for step in range(6):
        check_topk(B, ora, ctx, g, k, None, 9, step, expect_excluded=1)
        check_topk(B, ora, ctx, g, k, list(wl.geometric_probs(len(k))), 9, step, expect_excluded=0)
    if d > 5:
        gb = padded(torch.from_numpy(g_np).cuda().to(torch.bfloat16), 8)
        for step in range(3):
            check_topk(B, ora, ctx, gb, k, None, 10, step, expect_excluded=1)


def test_topk_candidate_overflow_takes_the_full_sweep_path(B, ora, ctx):
    # Nearly all entries share two magnitudes, so the boundary bins hold more keys than the candidate
    # buffer of this context (2^20 per worker): the digit passes and the band norms fall back to full sweeps.
    rng = np.random.default_rng(25)
    d = 1_300_000
    g_np = rng.choice(np.array([0.5, -0.5, 0.5000001, 3.0], dtype=np.float32), (2, d), p=[0.4, 0.3, 0.29, 0.01])
    g = to_dev(g_np)
    k = [100, 20_000, 400_000, 900_000, d]
    for step in range(3):
        check_topk(B, ora, ctx, g, k, None, 11, step, expect_excluded=1)
        check_topk(B, ora, ctx, g, k, list(wl.geometric_probs(len(k))), 11, step)


def test_fixed_p_brackets_hit_miss_and_restart(B, ora):
    """Fixed-p Top-k on fp32 reuses last call's boundary bins as brackets for the first sweep.  Every call must match
    the oracle whether the brackets hold (same distribution, next step), miss (the gradient is rescaled: the candidate
    pass runs after all) or do not exist yet (first call, new schedule)."""
    w = wl.shrink(wl.C3, 400_003, 3)
    k = wl.topk_schedule(w)
    L = len(k)
    c = B.mlmc_create(0, w.d, w.M, 32)
    try:
        sc = wl.scales(w, "cuda")
        one_level = np.full(L, 1e-9)
        one_level[3] = 1.0 - 1e-9 * (L - 1)                 # always level 3: the same two boundaries every step
        p = list(one_level)
        assert B.mlmc_read_bracket_stats(c) == (0, 0, 0)
        g0 = padded(wl.gradients(w, 0, "cuda", sc), 4)
        check_topk(B, ora, c, g0, k, p, w.seed, 0)
        assert B.mlmc_read_bracket_stats(c) == (0, 0, 3)    # first call: nothing stored yet
        for step in (1, 2, 3):
            g = padded(wl.gradients(w, step, "cuda", sc), 4)
            check_topk(B, ora, c, g, k, p, w.seed, step)
        hit, miss, none = B.mlmc_read_bracket_stats(c)
        assert none == 3 and hit + miss == 9 and hit >= 6   # fresh noise, same scales: the thresholds barely move
        g_big = padded(wl.gradients(w, 4, "cuda", sc) * 1000.0, 4)
        check_topk(B, ora, c, g_big, k, p, w.seed, 4)       # every threshold moved by ten binades: all brackets miss
        hit2, miss2, none2 = B.mlmc_read_bracket_stats(c)
        assert (hit2, miss2, none2) == (hit, miss + 3, none)
        check_topk(B, ora, c, g_big, k, p, w.seed, 5)       # and hold again on the rescaled gradient
        assert B.mlmc_read_bracket_stats(c)[0] == hit + 3
        k2 = list(k)
        k2[2] += 1                                          # another schedule: the stored bins are dropped
        check_topk(B, ora, c, g_big, k2, p, w.seed, 6)
        assert B.mlmc_read_bracket_stats(c)[2] == none + 3
        check_topk(B, ora, c, g0, k, list(wl.geometric_probs(L)), w.seed, 7)    # mixed levels, partly known
        check_topk(B, ora, c, g0, k, list(wl.geometric_probs(L)), w.seed, 8)
        ties = to_dev(np.random.default_rng(3).choice(np.array([0.5, -0.5, 0.25, 3.0], dtype=np.float32), (3, w.d)))
        check_topk(B, ora, c, ties, k, p, w.seed, 9)        # every key in two bins: brackets collect the whole row
        check_topk(B, ora, c, ties, k, p, w.seed, 10)
    finally:
        B.mlmc_destroy(c)


def test_topk_single_level_is_identity(B, ora, ctx):
    g_np = np.random.default_rng(23).standard_normal((3, 4097)).astype(np.float32)
    g = to_dev(g_np)
    out = B.TopkBuffers(3, 4097)
    B.mlmc_compress_topk(ctx, g, [4097], [1.0], 0, 0, out)
    dense = torch.empty(4097, dtype=torch.float32, device="cuda")
    assert B.mlmc_get_status(ctx) == 0
    assert out.count.tolist() == [4097] * 3 and out.level.tolist() == [0] * 3
    assert np.array_equal(out.val.cpu().numpy()[:, :4097], g_np)       # C^L(v) = v bit-exactly
    B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, 3, 4097, dense)
    check_topk(B, ora, ctx, g, [4097], None, 0, 0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_emission_reads_only_batches_that_can_hold_band_entries(B, ctx, dtype):
    """The emission lists, per worker, the batches (512 32-bit words; eight per tile) whose largest magnitude reaches
    the band's lower threshold.  The list must cover every batch that holds a band entry, stay within the row, and be
    the whole row for the last level (whose lower threshold is zero); a gradient with one loud layer lists few."""
    per_word = 2 if dtype == "bf16" else 1
    batch = 512 * per_word
    tile = 8 * batch
    M, d = 4, 40 * tile + 123
    rng = np.random.default_rng(5)
    g_np = (rng.standard_normal((M, d)) * 1e-3).astype(np.float32)
    g_np[:, 7 * tile:9 * tile] *= 1e3                       # one loud layer: tiles 7 and 8
    g = to_dev(g_np)
    if dtype == "bf16":
        g = padded(g.to(torch.bfloat16), 8)
    k = [64, 1024, d]
    out = B.TopkBuffers(M, d)
    batches_in_row = (d + tile - 1) // tile * 8
    for step, p in ((0, [0.98, 0.01, 0.01]), (1, [0.01, 0.98, 0.01]), (2, [0.005, 0.005, 0.99])):
        B.mlmc_compress_topk(ctx, g, k, p, 11, step, out)
        assert B.mlmc_get_status(ctx) == B.MLMC_OK
        listed, batches = B.mlmc_read_listed_tiles(ctx, M)
        assert batches == batches_in_row
        for m in range(M):
            n, lv = int(out.count[m]), int(out.level[m])
            touched = torch.unique((out.idx[m, :n].to(torch.int64) & 0xFFFFFFFF) // batch).numel()
            assert touched <= listed[m] <= batches
            if lv == 2:
                assert listed[m] == batches                 # everything below k_1: every batch can hold entries
            else:
                assert listed[m] <= 16                      # only batches of the loud layer (two tiles)


def test_many_workers_and_the_maximum_number_of_levels(B, ora):
    """M = 700 workers with L = 32 levels (the largest the ABI takes), Top-k adaptive and fixed p, and bit-wise:
    the per-worker tables of the emission and of the averaging kernels are sized by M."""
    M, d = 700, 9_001
    rng = np.random.default_rng(31)
    g_np = (rng.standard_normal((M, d)) * 10.0 ** rng.uniform(-2, 0, (M, 1))).astype(np.float32)
    g = to_dev(g_np)
    c = B.mlmc_create(0, d, M, 32)
    try:
        k = sorted(set(int(x) for x in np.geomspace(1, d, 32)))
        k += list(range(k[-1] - (32 - len(k)), k[-1]))      # pad with distinct values below d up to 32 levels
        k = sorted(set(k))[-32:]
        assert len(k) == 32 and k[-1] == d
        check_topk(B, ora, c, g, k, None, 5, 0, expect_excluded=2)
        check_topk(B, ora, c, g, k, list(wl.geometric_probs(32)), 5, 1, expect_excluded=2)
        check_bitwise(B, ora, c, g, list(range(1, 24)), None, 5, 2)
    finally:
        B.mlmc_destroy(c)


def test_level_probs(B, ora, ctx):
    w = wl.shrink(wl.C5A, 600_000, 4)
    k = wl.topk_schedule(w)
    L = len(k)
    g = wl.gradients(w, 2, "cuda")
    p_out = torch.zeros((4, L), dtype=torch.float64, device="cuda")
    d_out = torch.zeros((4, L), dtype=torch.float64, device="cuda")
    B.mlmc_level_probs(ctx, g, B.MLMC_TOPK, k, None, p_out, d_out)
    assert B.mlmc_get_status(ctx) == 0
    gh = wl.as_numpy_bits(g)
    for m in range(4):
        o = ora.topk(gh[m], k, None)
        assert np.allclose(p_out[m].cpu().numpy(), o.p, rtol=1e-11, atol=1e-15)
        assert np.allclose(d_out[m].cpu().numpy(), o.delta, rtol=1e-12, atol=0)
    # fixed p: probabilities are the normalised input, deltas still come from the data
    pf = list(wl.geometric_probs(L))
    B.mlmc_level_probs(ctx, g, B.MLMC_TOPK, k, pf, p_out, d_out)
    assert np.allclose(p_out.cpu().numpy(), np.tile(pf, (4, 1)), rtol=1e-15)
    assert np.allclose(d_out[0].cpu().numpy(), ora.topk(gh[0], k, None).delta, rtol=1e-12)
    # bit-wise
    b = [1, 2, 4, 8, 16, 23]
    p_b = torch.zeros((4, 6), dtype=torch.float64, device="cuda")
    d_b = torch.zeros((4, 6), dtype=torch.float64, device="cuda")
    B.mlmc_level_probs(ctx, g, B.MLMC_BITWISE, b, None, p_b, d_b)
    for m in range(4):
        o = ora.bitwise(gh[m], b, None)
        assert np.allclose(p_b[m].cpu().numpy(), o.p, rtol=1e-12, atol=1e-15)
        assert np.allclose(d_b[m].cpu().numpy(), o.delta, rtol=1e-13, atol=0)


def test_level_probs_bf16(B, ora, ctx):
    """mlmc_level_probs on bf16 input: Top-k (norms from the exact 2^15-bin counts) and bit-wise."""
    w = wl.shrink(wl.C4, 500_009, 3)
    k = wl.topk_schedule(w)
    L = len(k)
    g = padded(wl.gradients(w, 1, "cuda"), 8)
    p_out = torch.zeros((3, L), dtype=torch.float64, device="cuda")
    d_out = torch.zeros((3, L), dtype=torch.float64, device="cuda")
    B.mlmc_level_probs(ctx, g, B.MLMC_TOPK, k, None, p_out, d_out)
    assert B.mlmc_get_status(ctx) == 0
    gh = wl.as_numpy_bits(g)
    assert gh.dtype == np.uint16
    for m in range(3):
        o = ora.topk(gh[m], k, None)
        assert np.allclose(p_out[m].cpu().numpy(), o.p, rtol=1e-11, atol=1e-15)
        assert np.allclose(d_out[m].cpu().numpy(), o.delta, rtol=1e-12, atol=0)
    b = [1, 2, 4, 8, 16, 23]
    p_b = torch.zeros((3, 6), dtype=torch.float64, device="cuda")
    d_b = torch.zeros((3, 6), dtype=torch.float64, device="cuda")
    B.mlmc_level_probs(ctx, g, B.MLMC_BITWISE, b, None, p_b, d_b)
    for m in range(3):
        o = ora.bitwise(gh[m], b, None)
        assert np.allclose(p_b[m].cpu().numpy(), o.p, rtol=1e-12, atol=1e-15)
        assert np.allclose(d_b[m].cpu().numpy(), o.delta, rtol=1e-13, atol=0)


def test_c2_bitwise_all_steps(B, ora, ctx):
    w = wl.C2
    b, p = list(w.bits), list(wl.geometric_probs(6))
    for step in range(w.steps):
        g = wl.gradients(w, step, "cuda")
        check_bitwise(B, ora, ctx, g, b, p, w.seed, step)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bitwise_adaptive_ragged(B, ora, ctx, dtype):
    w = wl.shrink(wl.C5B, 333_337, 5)
    sc = wl.scales(w, "cuda")
    for step in range(4):
        g = wl.gradients(w, step, "cuda", sc)
        g = padded(g.to(torch.bfloat16), 8) if dtype == "bf16" else padded(g, 4)
        check_bitwise(B, ora, ctx, g, list(w.bits), None, w.seed, step)
        check_bitwise(B, ora, ctx, g, [1, 2, 3, 4, 5, 6, 7, 8], None, w.seed, step)    # unit schedule: 2 planes
        check_bitwise(B, ora, ctx, g, [23], None, w.seed, step)


def test_bitwise_degenerate(B, ora, ctx):
    z = to_dev(np.zeros((2, 1000), dtype=np.float32))
    check_bitwise(B, ora, ctx, z, [1, 2, 4], None, 0, 0)
    one = np.zeros((2, 1000), dtype=np.float32)
    one[0, 17] = -1e-40          # denormal maximum
    one[1, 999] = 5.0
    check_bitwise(B, ora, ctx, to_dev(one), [1, 2, 4, 23], None, 0, 1)
    check_bitwise(B, ora, ctx, to_dev(one), [1, 2, 4, 23], [0.25] * 4, 0, 2)


def test_device_errors_and_argument_checks(B, ctx):
    g = to_dev(np.random.default_rng(24).standard_normal((2, 5000)).astype(np.float32))
    k = [10, 100, 5000]
    out = B.TopkBuffers(2, 50)                    # too small for the top band
    hit = 0
    for step in range(12):
        B.mlmc_compress_topk(ctx, g, k, [0.2, 0.3, 0.5], 3, step, out)
        st = B.mlmc_get_status(ctx)
        lv, cnt = out.level.tolist(), out.count.tolist()
        if st == B.MLMC_ERR_CAPACITY:
            hit += 1
            assert any(l == -1 and c == 0 for l, c in zip(lv, cnt))
        else:
            assert st == 0 and all(c <= 50 for c in cnt)
    assert hit > 0
    assert B.mlmc_get_status(ctx) == 0            # sticky word was cleared
    bad = g.clone()
    bad[1, 4321] = float("nan")
    ok_out = B.TopkBuffers(2, 5000)
    B.mlmc_compress_topk(ctx, bad, k, None, 0, 0, ok_out)
    assert B.mlmc_get_status(ctx) == B.MLMC_ERR_NONFINITE
    assert ok_out.level.tolist()[1] == -1 and ok_out.count.tolist()[1] == 0 and ok_out.level.tolist()[0] >= 0
    bo = B.BitBuffers(2, 5000, 8)
    bad[1, 4321] = float("inf")
    B.mlmc_compress_bitwise(ctx, bad, [1, 2, 4, 8], None, 0, 0, bo)
    assert B.mlmc_get_status(ctx) == B.MLMC_ERR_NONFINITE and bo.level.tolist()[1] == -1
    dense = torch.zeros(5000, device="cuda")
    B.mlmc_aggregate(ctx, B.MLMC_BITWISE, bo, [1, 2, 4, 8], 2, 5000, dense)       # failed worker contributes nothing
    assert torch.isfinite(dense).all()
    for kk, pp, code in (([10, 100, 4999], None, B.MLMC_ERR_SCHEDULE), ([100, 10, 5000], None, B.MLMC_ERR_SCHEDULE),
                         (k, [0.5, 0.5, 0.0], B.MLMC_ERR_PROB), (k, [0.5, 0.4, 0.2], B.MLMC_ERR_PROB)):
        with pytest.raises(B.MlmcError) as e:
            B.mlmc_compress_topk(ctx, g, kk, pp, 0, 0, ok_out)
        assert e.value.code == code
    with pytest.raises(B.MlmcError) as e:
        B.mlmc_compress_bitwise(ctx, g, [1, 2, 24], None, 0, 0, bo)
    assert e.value.code == B.MLMC_ERR_SCHEDULE
    with pytest.raises(B.MlmcError) as e:         # misaligned gradient pointer
        B.mlmc_compress_topk(ctx, g[:1, 1:], [10, 4999], None, 0, 0, ok_out)
    assert e.value.code == B.MLMC_ERR_ARG


def test_run_to_run_determinism(B, ctx):
    w = wl.shrink(wl.C5A, 1_000_000, 4)
    k = wl.topk_schedule(w)
    g = wl.gradients(w, 0, "cuda")
    ref = None
    for _ in range(3):
        out = B.TopkBuffers(4, wl.max_band(k))
        dense = torch.empty(w.d, dtype=torch.float32, device="cuda")
        B.mlmc_compress_topk(ctx, g, k, None, 1, 2, out)
        B.mlmc_aggregate(ctx, B.MLMC_TOPK, out, None, 4, w.d, dense)
        assert B.mlmc_get_status(ctx) == 0
        n = out.count.tolist()
        snap = (out.level.tolist(), out.p_sel.tolist(), [out.idx[m, :n[m]].clone() for m in range(4)],
                [out.val[m, :n[m]].clone() for m in range(4)], dense.clone())
        if ref is not None:
            assert snap[0] == ref[0] and snap[1] == ref[1] and torch.equal(snap[4], ref[4])
            assert all(torch.equal(a, b) for a, b in zip(snap[2], ref[2]))
            assert all(torch.equal(a, b) for a, b in zip(snap[3], ref[3]))
        ref = snap


def test_two_contexts_side_by_side_on_two_streams(B, ctx):
    """A context serves one stream at a time; two contexts share nothing.  The Top-k and the bit-wise pipeline of a
    step, run side by side on two streams with a context each (as bench.py runs its two-variant workload), give
    bit for bit what they give one after the other on one stream (which the tests above compare with the oracle)."""
    w = wl.shrink(wl.C5A, 1_500_003, 4)
    k = wl.topk_schedule(w)
    bits = list(wl.C5B.bits)
    widths = [bits[0]] + [bits[i] - bits[i - 1] for i in range(1, len(bits))]
    sc = wl.scales(w, "cuda")
    other = B.mlmc_create(0, w.d, w.M, 32)
    side = torch.cuda.Stream(priority=-1)
    try:
        for step in range(4):
            g = padded(wl.gradients(w, step, "cuda", sc), 4)

            def run(side_by_side):
                mt, mb = B.TopkBuffers(w.M, wl.max_band(k)), B.BitBuffers(w.M, w.d, max(widths))
                dt = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
                db = torch.full((w.d,), float("nan"), dtype=torch.float32, device="cuda")
                main = torch.cuda.current_stream()
                if side_by_side:
                    fork = torch.cuda.Event()
                    fork.record(main)
                    side.wait_event(fork)
                    with torch.cuda.stream(side):
                        B.mlmc_compress_topk(other, g, k, None, w.seed, step, mt)
                        B.mlmc_aggregate(other, B.MLMC_TOPK, mt, None, w.M, w.d, dt)
                        done = torch.cuda.Event()
                        done.record(side)
                    B.mlmc_compress_bitwise(ctx, g, bits, None, w.seed, step, mb)
                    B.mlmc_aggregate(ctx, B.MLMC_BITWISE, mb, bits, w.M, w.d, db)
                    main.wait_event(done)
                else:
                    B.mlmc_compress_topk(ctx, g, k, None, w.seed, step, mt)
                    B.mlmc_aggregate(ctx, B.MLMC_TOPK, mt, None, w.M, w.d, dt)
                    B.mlmc_compress_bitwise(ctx, g, bits, None, w.seed, step, mb)
                    B.mlmc_aggregate(ctx, B.MLMC_BITWISE, mb, bits, w.M, w.d, db)
                torch.cuda.synchronize()
                assert B.mlmc_get_status(ctx) == 0 and B.mlmc_get_status(other) == 0
                n = mt.count.tolist()
                return (mt.level.tolist(), mt.p_sel.tolist(), n, [mt.idx[m, :n[m]].clone() for m in range(w.M)],
                        [mt.val[m, :n[m]].clone() for m in range(w.M)], dt, mb.level.tolist(), mb.p_sel.tolist(),
                        mb.gmax.clone(), [mb.planes[m, :1 + widths[l]].clone() for m, l in enumerate(mb.level.tolist())], db)

            a, b = run(False), run(True)
            assert a[0] == b[0] and a[1] == b[1] and a[2] == b[2] and a[6] == b[6] and a[7] == b[7]
            assert all(torch.equal(x, y) for x, y in zip(a[3], b[3])) and all(torch.equal(x, y) for x, y in zip(a[4], b[4]))
            assert torch.equal(a[5], b[5]) and torch.equal(a[8], b[8]) and torch.equal(a[10], b[10])
            assert all(torch.equal(x, y) for x, y in zip(a[9], b[9]))
    finally:
        B.mlmc_destroy(other)
