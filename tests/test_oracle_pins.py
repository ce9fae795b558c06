"""Pins for the CPU oracle: every check here is against something the paper or the mathematics
fixes (closed forms, brute force on tiny inputs, identities of Lemma 3.2 / 3.3 / 3.4, published
known-answer values), never against the oracle's own formula retyped.
"""
import itertools
import math

import numpy as np
import pytest

MASK = (1 << 64) - 1


# ----------------------------------------------------------------------------------------------
# counter RNG and the level draw
# ----------------------------------------------------------------------------------------------
def _splitmix_out(z):
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK
    return z ^ (z >> 31)


G = 0x9E3779B97F4A7C15


def test_splitmix_published_vectors():
    # SplitMix64 seeded with 0: the first three outputs of the published generator.
    assert _splitmix_out(G) == 0xE220A8397B1DCDAF
    assert _splitmix_out((2 * G) & MASK) == 0x6E789E6AA1B965F4
    assert _splitmix_out((3 * G) & MASK) == 0x06C45D188009454F


def test_hash_is_three_chained_splitmix_rounds(ora):
    rng = np.random.default_rng(5)
    cases = [(0, 0, 0), (1, 2, 3), (MASK, MASK, MASK)] + [tuple(int(x) for x in rng.integers(0, 2**63, 3)) for _ in range(50)]
    for seed, step, worker in cases:
        h = _splitmix_out((seed + G) & MASK)
        h = _splitmix_out((h + step + G) & MASK)
        h = _splitmix_out((h + worker + G) & MASK)
        assert ora.hash64(seed, step, worker) == h
        assert ora.uniform(seed, step, worker) == (h >> 11) * 2.0**-53
    # with seed 0 the first round is the published first output
    h = _splitmix_out((0xE220A8397B1DCDAF + 0 + G) & MASK)
    assert ora.hash64(0, 0, 0) == _splitmix_out((h + G) & MASK)


def test_uniform_is_uniform(ora):
    n, bins = 200_000, 64
    u = np.array([ora.uniform(9, s, w) for s in range(n // 8) for w in range(8)])
    assert u.min() >= 0.0 and u.max() < 1.0
    cnt = np.bincount((u * bins).astype(int), minlength=bins)
    chi2 = ((cnt - n / bins) ** 2 / (n / bins)).sum()
    assert chi2 < 63 + 6 * math.sqrt(2 * 63)  # ~6 sigma of chi^2_63
    assert abs(u.mean() - 0.5) < 5 / math.sqrt(12 * n)
    # neighbouring counters are uncorrelated
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 5 / math.sqrt(n)


def test_draw_worked_example(ora):
    p = [0.5, 0.25, 0.25]
    assert ora.draw(p, 0.6) == (1, pytest.approx(0.1))
    assert ora.draw(p, 0.0)[0] == 0
    assert ora.draw(p, 0.5)[0] == 1          # strict u < cdf
    assert ora.draw(p, 0.75)[0] == 2
    assert ora.draw(p, 1 - 2.0**-53)[0] == 2
    assert ora.draw([1.0], 0.3) == (0, math.inf)
    # zero-probability levels are never drawn, also when they come last
    assert ora.draw([0.0, 0.5, 0.0, 0.5, 0.0], 0.99999)[0] == 3
    assert ora.draw([0.0, 0.5, 0.0, 0.5, 0.0], 0.0)[0] == 1
    assert ora.draw([0.0, 0.5, 0.0, 0.5, 0.0], 0.5)[0] == 3


def test_draw_interval_and_frequencies(ora):
    rng = np.random.default_rng(1)
    p = rng.random(9)
    p /= p.sum()
    tail = np.cumsum(p[::-1])[::-1]            # second summation order: 1 - tail
    counts = np.zeros(9)
    n = 60_000
    for t in range(n):
        u = ora.uniform(3, t, 0)
        lv, margin = ora.draw(p, u)
        counts[lv] += 1
        if margin > 1e-9:
            lo = 0.0 if lv == 0 else 1.0 - tail[lv]
            hi = 1.0 if lv == 8 else 1.0 - tail[lv + 1]
            assert lo <= u < hi
    assert np.all(np.abs(counts / n - p) < 5 * np.sqrt(p * (1 - p) / n))


# ----------------------------------------------------------------------------------------------
# total order, bands, Top-k identities
# ----------------------------------------------------------------------------------------------
def _brute_rank(g):
    a = np.abs(g.astype(np.float64))
    d = len(g)
    r = np.zeros(d, dtype=int)
    for i in range(d):
        r[i] = sum(1 for j in range(d) if a[j] > a[i] or (a[j] == a[i] and j < i))
    perm = np.empty(d, dtype=int)
    perm[r] = np.arange(d)
    return perm


def test_rank_brute_force_with_ties(ora):
    rng = np.random.default_rng(2)
    for d in (1, 2, 5, 12):
        for _ in range(20):
            g = rng.integers(-3, 4, d).astype(np.float32) * 0.5   # many ties, +-0 included
            g[rng.random(d) < 0.2] *= -1.0
            assert np.array_equal(ora.rank(g), _brute_rank(g))
    g = np.array([0.0, -0.0, 1e-45, -1e-45, 1.0, -1.0], dtype=np.float32)  # zeros, denormals
    assert list(ora.rank(g)) == [4, 5, 2, 3, 0, 1]


def test_rank_bf16_matches_widened_fp32(ora):
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 2**16, 500).astype(np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]                         # finite only
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(ora.rank(bits), ora.rank(wide))
    assert np.array_equal(ora.rank(bits), _brute_rank(wide))


def _all_levels(ora, g, k, p):
    return [ora.topk(g, k, p=p, force_level=l) for l in range(len(k))]


@pytest.mark.parametrize("adaptive", [False, True])
def test_bands_partition_and_unbiasedness(ora, adaptive):
    rng = np.random.default_rng(4)
    d = 257
    g = (rng.standard_normal(d) * 10.0 ** rng.uniform(-3, 0, d)).astype(np.float32)
    g[::7] = g[3]                                                   # ties across band edges
    k = [1, 2, 2, 9, 40, 41, 200, d]
    L = len(k)
    p = None if adaptive else rng.dirichlet(np.ones(L))
    msgs = _all_levels(ora, g, k, p)
    perm = _brute_rank(g)
    seen = np.zeros(d, dtype=int)
    mean32 = np.zeros(d)
    mean64 = np.zeros(d)
    for l, m in enumerate(msgs):
        lo = k[l - 1] if l else 0
        assert m.idx.size == k[l] - lo                              # band size
        assert np.all(np.diff(m.idx.astype(np.int64)) > 0)          # ascending, unique
        assert set(m.idx.tolist()) == set(perm[lo:k[l]].tolist())   # ranks (k_{l-1}, k_l]
        seen[m.idx] += 1
        assert m.p_sel == m.p[l]
        if m.p_sel > 0:
            assert np.array_equal(m.val, (g[m.idx].astype(np.float64) / m.p_sel).astype(np.float32))
        mean32[m.idx] += m.p_sel * m.val.astype(np.float64)
        mean64[m.idx] += m.p_sel * (g[m.idx].astype(np.float64) / m.p_sel) if m.p_sel > 0 else 0.0
    assert np.all(seen == 1)                                        # telescoping: bands partition [d]
    assert abs(msgs[0].p.sum() - 1.0) < 1e-14
    # Lemma 3.2: sum_l p_l * est_l = C^L(g) = g
    assert np.allclose(mean64, g.astype(np.float64), rtol=1e-12, atol=0)
    assert np.allclose(mean32, g.astype(np.float64), rtol=2.0**-23, atol=0)   # fp32 message values


def test_top_level_is_identity(ora):
    rng = np.random.default_rng(6)
    g = rng.standard_normal(100).astype(np.float32)
    m = ora.topk(g, [100], p=[1.0])
    assert m.level == 0 and m.p_sel == 1.0
    assert np.array_equal(m.idx, np.arange(100)) and np.array_equal(m.val, g)   # C^L(v) = v bit-exactly


def test_unit_schedule_is_lth_largest_entry_and_importance_sampling(ora):
    # Sec. 3.2: with k_l = l the residual is the l-th largest entry; Sec. 3.3: MLMC = importance sampling,
    # so the adaptive second moment (sum Delta)^2 equals ||g||_1^2.
    rng = np.random.default_rng(7)
    d = 23
    g = rng.standard_normal(d).astype(np.float32)
    k = list(range(1, d + 1))
    order = np.argsort(-np.abs(g), kind="stable")
    msgs = _all_levels(ora, g, k, None)
    for l, m in enumerate(msgs):
        assert m.idx.tolist() == [order[l]]
        assert m.delta[l] == pytest.approx(abs(float(g[order[l]])), rel=1e-15)
    second = sum(m.p_sel * float(np.sum(m.val.astype(np.float64) ** 2)) for m in msgs)
    l1 = float(np.sum(np.abs(g.astype(np.float64))))
    assert second == pytest.approx(l1**2, rel=1e-6)
    assert np.sum(msgs[0].delta) ** 2 == pytest.approx(l1**2, rel=1e-13)


def test_contraction_bound(ora):
    # ||C^l(v) - v||^2 <= (1 - k_l/d) ||v||^2, with equality when |v| is constant (Sec. 3.2).
    rng = np.random.default_rng(8)
    d = 120
    k = [5, 17, 60, 119, 120]
    for const in (False, True):
        g = rng.standard_normal(d).astype(np.float32)
        if const:
            g = (np.sign(g) * 0.37).astype(np.float32)
        g64 = g.astype(np.float64)
        kept = np.zeros(d, dtype=bool)
        for l, m in enumerate(_all_levels(ora, g, k, None)):
            kept[m.idx] = True                                      # C^l(g) = union of bands 0..l
            dist = float(np.sum(g64[~kept] ** 2))
            bound = (1 - k[l] / d) * float(np.sum(g64**2))
            assert dist <= bound * (1 + 1e-12)
            if const:
                assert dist == pytest.approx(bound, rel=1e-12, abs=1e-300)
            # Eq. 7: alpha^l = ||C^l(v)||^2 / ||v||^2, and Delta_l^2 = (alpha^l - alpha^{l-1}) ||v||^2
        assert kept.all()


def test_second_moment_and_adaptive_optimum(ora):
    rng = np.random.default_rng(9)
    d = 300
    g = (rng.standard_normal(d) * 10.0 ** rng.uniform(-2, 0, d)).astype(np.float32)
    g64 = g.astype(np.float64)
    k = [3, 10, 30, 100, 300]
    ad = _all_levels(ora, g, k, None)
    delta = ad[0].delta
    # Delta_l is the l2 norm of the band (definition under Lemma 3.4), checked against the bands themselves
    for l, m in enumerate(ad):
        assert delta[l] == pytest.approx(math.sqrt(float(np.sum(g64[m.idx] ** 2))), rel=1e-14)
    assert np.allclose(ad[0].p, delta / delta.sum(), rtol=1e-15)
    # App. D: E||g~||^2 = sum_l Delta_l^2 / p_l for any p; = (sum Delta)^2 at the optimum
    def second_moment(msgs):
        return sum(m.p_sel * float(np.sum((g64[m.idx] / m.p_sel) ** 2)) for m in msgs)
    assert second_moment(ad) == pytest.approx(delta.sum() ** 2, rel=1e-12)
    # variance (sum Delta)^2 - ||v||^2 >= 0
    assert delta.sum() ** 2 >= np.sum(g64**2)
    for _ in range(20):
        p = rng.dirichlet(np.ones(len(k)))
        fx = _all_levels(ora, g, k, p)
        assert np.allclose(fx[0].delta, delta, rtol=1e-15)
        sm = second_moment(fx)
        assert sm == pytest.approx(float(np.sum(delta**2 / fx[0].p)), rel=1e-12)
        assert sm >= delta.sum() ** 2 * (1 - 1e-12)                 # optimality of the adaptive p


def test_exponential_decay_closed_forms(ora):
    # Assumption 3.5 / Lemma 3.6 and App. E: |v(j)| = a exp(-r j / 2) on the sorted vector,
    # uniform schedule k_l = s l (s-Top-k), s L = d.
    rng = np.random.default_rng(10)
    d, s, r, a = 4096, 64, 0.01, 3.0
    L = d // s
    mags = a * np.exp(-0.5 * r * np.arange(d))
    pi = rng.permutation(d)
    g = np.empty(d, dtype=np.float32)
    g[pi] = (mags * rng.choice([-1.0, 1.0], d)).astype(np.float32)
    k = [s * (l + 1) for l in range(L)]
    m = ora.topk(g, k, None)
    a32 = float(np.float32(a))
    norm2 = a**2 * (1 - math.exp(-r * d)) / (1 - math.exp(-r))
    assert float(np.sum(g.astype(np.float64) ** 2)) == pytest.approx(norm2, rel=1e-6)
    lvl = np.arange(1, L + 1)
    delta2 = a**2 * np.exp(-r * s * (lvl - 1)) * (1 - math.exp(-r * s)) / (1 - math.exp(-r))
    assert np.allclose(m.delta**2, delta2, rtol=2e-6)
    var = m.delta.sum() ** 2 - float(np.sum(g.astype(np.float64) ** 2))
    exact = norm2 * ((1 - math.exp(-r * s)) / (1 - math.exp(-r * d))
                     * ((1 - math.exp(-0.5 * r * d)) / (1 - math.exp(-0.5 * r * s))) ** 2 - 1)
    assert var == pytest.approx(exact, rel=1e-5)
    assert var == pytest.approx(norm2 * (4 / (r * s) - 1), rel=0.10)   # O(1/(r s)) regime: r d >> 1, r s <= 1
    assert a32 > 0


def test_monte_carlo_mean(ora):
    rng = np.random.default_rng(11)
    d = 16
    g = (rng.standard_normal(d) * 10.0 ** rng.uniform(-1, 0, d)).astype(np.float32)
    k = [1, 2, 4, 8, 16]
    for p in (None, np.array([0.4, 0.3, 0.15, 0.1, 0.05])):
        N = 30_000
        acc = np.zeros(d)
        levels = np.zeros(len(k))
        for t in range(N):
            m = ora.topk(g, k, p=p, seed=77, step=t, worker=5)
            acc[m.idx] += m.val
            levels[m.level] += 1
        ref = ora.topk(g, k, p=p)
        # per-coordinate variance from the enumerated second moment: coordinate i lives in one band l(i)
        var = np.zeros(d)
        for l in range(len(k)):
            mm = ora.topk(g, k, p=p, force_level=l)
            var[mm.idx] = (g[mm.idx].astype(np.float64) ** 2) * (1 / mm.p_sel - 1)
        assert np.all(np.abs(acc / N - g) <= 4.5 * np.sqrt(var / N) + 1e-7)
        assert np.all(np.abs(levels / N - ref.p) < 5 * np.sqrt(ref.p * (1 - ref.p) / N) + 1e-12)


def test_topk_argument_errors(ora):
    g = np.ones(8, dtype=np.float32)
    for k, p, code in (([4, 7], None, ora.ERR_SCHEDULE), ([5, 4, 8], None, ora.ERR_SCHEDULE),
                       ([4, 8], [1.0, 0.0], ora.ERR_PROB), ([4, 8], [0.7, 0.7], ora.ERR_PROB)):
        with pytest.raises(ora.OracleError) as e:
            ora.topk(g, k, p=p)
        assert e.value.code == code
    bad = g.copy()
    bad[3] = np.nan
    with pytest.raises(ora.OracleError) as e:
        ora.topk(bad, [8], None)
    assert e.value.code == ora.ERR_NONFINITE


def test_zero_gradient_and_empty_bands(ora):
    z = np.zeros(10, dtype=np.float32)
    m = ora.topk(z, [3, 10], None, seed=1)
    assert m.level == 0 and m.p_sel == 1.0 and m.idx.tolist() == [0, 1, 2] and not m.val.any()
    g = np.arange(1, 11, dtype=np.float32)
    ms = _all_levels(ora, g, [4, 4, 10], None)                       # k_l = k_{l-1}: empty band, p = 0
    assert ms[1].idx.size == 0 and ms[1].p[1] == 0.0 and ms[1].delta[1] == 0.0
    assert {ora.topk(g, [4, 4, 10], None, step=t).level for t in range(200)} == {0, 2}


# ----------------------------------------------------------------------------------------------
# fixed-point bit-wise compressor (Sec. 3.1, Lemma 3.3, App. C)
# ----------------------------------------------------------------------------------------------
def test_fixed_point_codes_hand_example(ora):
    g = np.array([1.0, 0.5, 0.25, -0.75, 0.0, -0.0, 0.3], dtype=np.float32)
    gmax, q = ora.fixed_point_codes(g, 4)
    assert gmax == 1.0
    assert q.tolist() == [15, 8, 4, 12, 0, 0, 4]      # |e| = 1 clamps to 2^B - 1; 0.3 * 16 = 4.8 -> 4
    gmax, q = ora.fixed_point_codes(g * np.float32(8.0), 4)          # scale invariance by powers of two
    assert gmax == 8.0 and q.tolist() == [15, 8, 4, 12, 0, 0, 4]
    gmax, q = ora.fixed_point_codes(np.zeros(5, dtype=np.float32), 23)
    assert gmax == 0.0 and not q.any()


def test_fixed_point_unit_schedule_lemma_3_3(ora):
    rng = np.random.default_rng(12)
    d, B = 200, 12
    g = (rng.standard_t(3, d) * 1e-2).astype(np.float32)
    b = list(range(1, B + 1))
    p = np.array([2.0 ** -(l + 1) / (1 - 2.0**-B) for l in range(B)])   # Lemma 3.3 with B bits
    gmax, q = ora.fixed_point_codes(g, B)
    msgs = [ora.bitwise(g, b, p=p, force_level=l) for l in range(B)]
    sign = np.where(np.signbit(g), -1.0, 1.0)
    mean = np.zeros(d)
    second = np.zeros(d)
    for l, m in enumerate(msgs):
        assert m.planes.shape[0] == 2                                # one information bit + one sign bit
        est = ora.bitwise_decode(m.planes, d, b, l, m.gmax, m.p_sel)
        bit = (q >> (B - 1 - l)) & 1
        assert np.array_equal(est, sign * bit * 2.0 ** -(l + 1) * float(np.float32(gmax)) / m.p_sel)
        mean += m.p_sel * est
        second += m.p_sel * (est / gmax) ** 2
    e_q = q * 2.0**-B
    # App. C: per-entry second moment = (1 - 2^-B) |e|, for the normalised entry
    assert np.allclose(second, (1 - 2.0**-B) * e_q, rtol=1e-12, atol=0)
    # unbiased for the B-bit code Q_B(g), which is within 2^-B gmax of g
    QB = sign * e_q * gmax
    assert np.allclose(mean, QB, rtol=1e-12, atol=0)
    assert np.all(np.abs(QB - g) <= 2.0**-B * gmax * (1 + 2.0**-23))
    # sigma^2_comp = (1 - 2^-B) ||v||_1 - ||v||^2 for the normalised code vector
    assert second.sum() - np.sum(e_q**2) == pytest.approx((1 - 2.0**-B) * e_q.sum() - np.sum(e_q**2), rel=1e-12)


def test_fixed_point_multibit_levels(ora):
    rng = np.random.default_rng(13)
    d = 333                                                            # ragged last word
    g = (rng.standard_t(3, d) * 1e-2).astype(np.float32)
    b = [1, 2, 4, 8, 16, 23]
    gmax, q = ora.fixed_point_codes(g, 23)
    sign = np.where(np.signbit(g), -1.0, 1.0)
    for p in (None, np.array([2.0**-l for l in range(6)]) / sum(2.0**-l for l in range(6))):
        msgs = [ora.bitwise(g, b, p=p, force_level=l) for l in range(6)]
        mean = np.zeros(d)
        trunc = np.zeros(d)
        for l, m in enumerate(msgs):
            w = b[l] - (b[l - 1] if l else 0)
            assert m.planes.shape == (1 + w, (d + 31) // 32)
            assert m.planes[:, -1].max() < 2 ** (d % 32)               # tail bits beyond d are zero
            est = ora.bitwise_decode(m.planes, d, b, l, m.gmax, m.p_sel)
            mean += m.p_sel * est
            # level-l compressor = code truncated to b_l bits: distortion <= 2^-b_l per normalised entry
            trunc += m.p_sel * est
            assert np.all(np.abs(np.abs(trunc) - q * 2.0**-23 * gmax) <= 2.0 ** -b[l] * gmax * (1 + 1e-12))
            # exact integer field energy
            f = (q >> (23 - b[l])) & ((1 << w) - 1)
            assert int(m.S[l]) == int(np.sum(f.astype(np.uint64) ** 2))
            assert m.delta[l] == pytest.approx(gmax * 2.0 ** -b[l] * math.sqrt(float(m.S[l])), rel=1e-15)
        assert np.allclose(mean, sign * q * 2.0**-23 * gmax, rtol=1e-12, atol=0)   # telescopes to Q_B(g)
        if p is None:
            assert np.allclose(msgs[0].p, msgs[0].delta / msgs[0].delta.sum(), rtol=1e-15)


def test_bitwise_zero_and_errors(ora):
    z = np.zeros(40, dtype=np.float32)
    m = ora.bitwise(z, [1, 2, 4], None)
    assert m.level == 0 and m.gmax == 0.0 and not m.planes.any()
    for b in ([2, 2], [3, 1], [1, 24]):
        with pytest.raises(ora.OracleError) as e:
            ora.bitwise(np.ones(4, dtype=np.float32), b, None)
        assert e.value.code == ora.ERR_SCHEDULE


# ----------------------------------------------------------------------------------------------
# server aggregation (Alg. 2, "Server aggregates")
# ----------------------------------------------------------------------------------------------
def test_aggregate_topk(ora):
    rng = np.random.default_rng(14)
    d = 500
    g = rng.standard_normal(d).astype(np.float32)
    m = ora.topk(g, [d], p=[1.0])
    out, scale = ora.aggregate_topk([(m.idx, m.val)], d)
    assert np.array_equal(out, g.astype(np.float64)) and np.array_equal(scale, np.abs(g).astype(np.float64))
    M = 5
    k = [7, 50, 200, d]
    msgs, dense = [], np.zeros(d)
    for w in range(M):
        gw = rng.standard_normal(d).astype(np.float32)
        mw = ora.topk(gw, k, None, seed=2, step=1, worker=w)
        msgs.append((mw.idx, mw.val))
        dense[mw.idx] += mw.val.astype(np.float64)
    out, scale = ora.aggregate_topk(msgs, d)
    assert np.allclose(out, dense / M, rtol=1e-15, atol=0)
    # linearity: aggregating a message twice doubles its share
    out2, _ = ora.aggregate_topk(msgs + msgs, d)
    assert np.allclose(out2, out, rtol=1e-15, atol=0)


def test_aggregate_scale_is_the_mean_of_absolute_terms_hand_example(ora):
    """Alg. 2 "Server aggregates" on hand-written messages: M = 3 workers, overlapping coordinates, mixed signs.
    The expected mean and the expected tolerance scale (1/M) sum_m |term_m| are typed in by hand (exact in binary)."""
    d = 6
    msgs = [(np.array([0, 2, 5], dtype=np.uint32), np.array([1.5, -3.0, 0.75], dtype=np.float32)),
            (np.array([2, 3], dtype=np.uint32), np.array([3.0, -6.0], dtype=np.float32)),
            (np.array([0, 2, 3], dtype=np.uint32), np.array([-4.5, 1.5, -1.5], dtype=np.float32))]
    out, scale = ora.aggregate_topk(msgs, d)
    assert out.tolist() == [-1.0, 0.0, 0.5, -2.5, 0.0, 0.25]
    assert scale.tolist() == [2.0, 0.0, 2.5, 2.5, 0.0, 0.25]
    # the scale is a mean, not a sum: the same three messages sent twice (M = 6) leave it unchanged
    out6, scale6 = ora.aggregate_topk(msgs + msgs, d)
    assert out6.tolist() == out.tolist() and scale6.tolist() == scale.tolist()


def test_aggregate_bitwise_scale_hand_example(ora):
    """Bit-plane messages typed in by hand: b = (1, 3), d = 3, M = 2.  Worker 0 sends level 1 (a 2-bit field) with
    gmax 4 and p 1/2, worker 1 sends level 0 (a 1-bit field) with gmax 2 and p 1/4.  A residual entry is
    sign f 2^-b_l gmax / p (Sec. 3.1), so the terms are (3, -1, 0) and (-4, 0, 4); mean and scale follow by hand."""
    class Msg:
        pass
    a, c = Msg(), Msg()
    # worker 0: fields (3, 1, 0) -> planes: sign 0b010, msb 0b001, lsb 0b011; unit = 2^-3 * 4 / (1/2) = 1
    a.planes = np.array([[0b010], [0b001], [0b011]], dtype=np.uint32)
    a.gmax, a.level, a.p_sel = 4.0, 1, 0.5
    # worker 1: fields (1, 0, 1) -> planes: sign 0b001, bit 0b101; unit = 2^-1 * 2 / (1/4) = 4
    c.planes = np.array([[0b001], [0b101]], dtype=np.uint32)
    c.gmax, c.level, c.p_sel = 2.0, 0, 0.25
    out, scale = ora.aggregate_bitwise([a, c], [1, 3], 3)
    assert out.tolist() == [-0.5, -0.5, 2.0]
    assert scale.tolist() == [3.5, 0.5, 2.0]


def test_aggregate_bitwise(ora):
    rng = np.random.default_rng(15)
    d, M = 130, 4
    b = [1, 2, 4, 8]
    msgs, dense = [], np.zeros(d)
    for w in range(M):
        gw = rng.standard_normal(d).astype(np.float32)
        mw = ora.bitwise(gw, b, None, seed=3, step=0, worker=w)
        msgs.append(mw)
        dense += ora.bitwise_decode(mw.planes, d, b, mw.level, mw.gmax, mw.p_sel)
    out, scale = ora.aggregate_bitwise(msgs, b, d)
    assert np.allclose(out, dense / M, rtol=1e-15, atol=0)
    assert np.all(scale >= np.abs(out) - 1e-15)


def test_rng_golden_file_matches_oracle(ora):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "rng_kat.txt")
    rows = [ln.split() for ln in open(path) if not ln.startswith("#")]
    assert len(rows) == 16
    for s, t, w, h, u in rows:
        assert ora.hash64(int(s), int(t), int(w)) == int(h, 16)
        assert ora.uniform(int(s), int(t), int(w)) == float.fromhex(u)
