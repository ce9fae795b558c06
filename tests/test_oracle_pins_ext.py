"""Pins of the oracle's floating-point bit-wise, s-Top-k and RTN functions against what the paper and the
mathematics fix (no GPU).  Each check uses something other than the oracle's own formula: frexp / floor
arithmetic in fp64 for the mantissa truncation, closed forms of App. B, a brute-force sort for the segments,
exact rational arithmetic for the RTN grid, and hand-typed messages.
"""
from fractions import Fraction

import numpy as np
import pytest

F32_BITS = 23


def _trunc_by_frexp(x: np.ndarray, keep: int) -> np.ndarray:
    """sign 2^E floor(|x| / 2^E 2^keep) / 2^keep for normal fp32 x, in exact fp64 arithmetic (App. B, first display)."""
    x = x.astype(np.float64)
    mant, exp = np.frexp(np.abs(x))           # |x| = mant 2^exp, mant in [0.5, 1)
    e = exp - 1                               # |x| = (2 mant) 2^e with 2 mant in [1, 2)
    frac = 2.0 * mant
    kept = np.floor(np.ldexp(frac, keep)) / (1 << keep)
    return np.sign(x) * np.ldexp(kept, e)


# ----------------------------------------------------------------------------------------------
# floating-point compressor and its MLMC estimate (Sec. 2.2, App. B)
# ----------------------------------------------------------------------------------------------
def test_float_compressor_is_mantissa_truncation(ora):
    rng = np.random.default_rng(40)
    g = (rng.standard_normal(4000) * 10.0 ** rng.uniform(-6, 3, 4000)).astype(np.float32)
    for keep in (0, 1, 2, 5, 11, 22, 23):
        assert np.array_equal(ora.float_compress(g, keep), _trunc_by_frexp(g, keep))
    assert np.array_equal(ora.float_compress(g, 23), g.astype(np.float64))        # Def. 3.1: top level = identity
    # contraction of App. B: |C^l(e) - e| < 2^-l 2^E <= 2^-l |e|
    for keep in (1, 4, 9):
        err = np.abs(ora.float_compress(g, keep) - g.astype(np.float64))
        assert np.all(err <= np.ldexp(np.abs(g).astype(np.float64), -keep))


def test_float_compressor_zero_subnormal_and_bf16(ora):
    g = np.array([0.0, -0.0, 1e-45, -3e-41, 1.17549435e-38, -1.5], dtype=np.float32)
    c0 = ora.float_compress(g, 0)
    assert c0[0] == 0.0 and c0[1] == 0.0 and c0[2] == 0.0 and c0[3] == 0.0        # exponent field 0: no leading one
    assert c0[4] == float(np.float32(1.17549435e-38)) and c0[5] == -1.0
    assert np.array_equal(ora.float_compress(g, 23), g.astype(np.float64))
    # subnormals: truncation of the integer mantissa (scale 2^-149)
    m = int(np.float32(3e-41).view(np.uint32))
    assert ora.float_compress(g, 10)[3] == -float((m >> 13) << 13) * 2.0 ** -149
    bf = np.array([0x3FC0, 0xBF81, 0x0001, 0x7F7F], dtype=np.uint16)               # 1.5, -1.0078125, tiny, max
    wide = (bf.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(ora.float_compress(bf, 7), wide.astype(np.float64))
    assert np.array_equal(ora.float_compress(bf, 3), _trunc_by_frexp(wide, 3) * (np.abs(wide) >= 1e-38))


def test_floatbits_hand_example(ora):
    """e = -1.75 = -(1 + 1/2 + 1/4): mantissa digits 1, 1, 0, ...  Unit schedule on the first three digits would need
    F = 23 levels; here the schedule (1, 2, 23) has fields of 1, 1 and 21 digits.  Level 0: residual 1/2 -> estimate
    -(1 + (1/2)/p_0); level 1: residual 1/4; level 2: residual 0 -> the base alone.  Message words typed by hand."""
    g = np.array([-1.75, 0.5], dtype=np.float32)
    mb = [1, 2, 23]
    p = [0.5, 0.25, 0.25]
    m0 = ora.floatbits(g, mb, p, force_level=0)
    assert m0.expo.tolist() == [127, 126]
    assert m0.planes.tolist() == [[0b01], [0b01]]                  # sign plane; first mantissa digit
    assert m0.est.tolist() == [-(1.0 + 0.5 / 0.5), 0.5]
    m1 = ora.floatbits(g, mb, p, force_level=1)
    assert m1.planes.tolist() == [[0b01], [0b01]] and m1.est.tolist() == [-(1.0 + 0.25 / 0.25), 0.5]
    m2 = ora.floatbits(g, mb, p, force_level=2)
    assert m2.planes.shape == (22, 1) and not m2.planes[1:].any() and m2.est.tolist() == [-1.0, 0.5]


def test_floatbits_unbiased_by_enumeration_and_telescoping(ora):
    rng = np.random.default_rng(41)
    g = (rng.standard_normal(3000) * 10.0 ** rng.uniform(-4, 2, 3000)).astype(np.float32)
    g[:4] = [0.0, -0.0, 1e-44, -2.0]
    for mb, p in (([1, 2, 4, 8, 16, 23], None), (list(range(1, 24)), None), ([3, 23], [0.3, 0.7])):
        base = ora.float_compress(g, 0)
        tele = base.copy()
        mean = np.zeros(g.size)
        for l in range(len(mb)):
            m = ora.floatbits(g, mb, p, force_level=l)
            lo = mb[l - 1] if l else 0
            res = ora.float_compress(g, mb[l]) - ora.float_compress(g, lo)        # C^l - C^{l-1}, exact in fp64
            assert np.all(np.abs(m.est - (base + res / m.p_sel)) <= 4e-16 * np.abs(m.est))
            tele += ora.float_compress(g, mb[l]) - ora.float_compress(g, lo)
            mean += m.p_sel * m.est
            assert np.allclose(ora.floatbits_decode(m.expo, m.planes, g.size, mb, l, m.p_sel), m.est, rtol=1e-15, atol=0)
        assert np.array_equal(tele, g.astype(np.float64))            # telescoping to g exactly (C^L = identity)
        assert np.allclose(mean, g.astype(np.float64), rtol=1e-14, atol=0)   # Lemma 3.2 (sum_l p_l = 1)


def test_floatbits_lemma_probabilities_and_second_moment(ora):
    """App. B: for the unit schedule p^l = 2^-l / (1 - 2^-F) (l = 1..F), and the second moment of the residual part of
    an entry is 2^E (1 - 2^-F) (|e| - 2^E)."""
    rng = np.random.default_rng(42)
    g = (rng.standard_normal(500) * 10.0 ** rng.uniform(-3, 3, 500)).astype(np.float32)
    mb = list(range(1, 24))
    m = ora.floatbits(g, mb, None, force_level=0)
    want = np.ldexp(1.0, -np.arange(1, 24)) / (1.0 - 2.0 ** -23)
    assert np.allclose(m.p, want, rtol=1e-15)
    base = ora.float_compress(g, 0)
    second = np.zeros(g.size)
    for l in range(23):
        ml = ora.floatbits(g, mb, None, force_level=l)
        second += ml.p_sel * (ml.est - base) ** 2
    two_e = np.abs(base)
    closed = two_e * (1.0 - 2.0 ** -23) * (np.abs(g.astype(np.float64)) - two_e)
    assert np.allclose(second, closed, rtol=1e-12, atol=0)
    # general schedule: p_l proportional to the largest residual of the level, 2^-m_{l-1} - 2^-m_l
    m6 = ora.floatbits(g, [1, 2, 4, 8, 16, 23], None, force_level=0)
    w = np.array([1 - 2.0 ** -1, 2.0 ** -1 - 2.0 ** -2, 2.0 ** -2 - 2.0 ** -4, 2.0 ** -4 - 2.0 ** -8,
                  2.0 ** -8 - 2.0 ** -16, 2.0 ** -16 - 2.0 ** -23])
    assert np.allclose(m6.p, w / w.sum(), rtol=1e-15)


def test_floatbits_message_size_draw_and_errors(ora):
    g = np.random.default_rng(43).standard_normal(100).astype(np.float32)
    m = ora.floatbits(g, list(range(1, 24)), None, seed=5, step=6, worker=7)
    assert m.planes.shape == (2, 4) and m.expo.size == 100          # 1 sign + 8 exponent + 1 mantissa bit per entry
    assert m.u == ora.uniform(5, 6, 7) and ora.draw(m.p, m.u)[0] == m.level
    for mb in ([1, 1, 23], [2, 1, 23], [1, 2, 22], [1, 24]):
        with pytest.raises(ora.OracleError) as e:
            ora.floatbits(g, mb, None)
        assert e.value.code == ora.ERR_SCHEDULE
    with pytest.raises(ora.OracleError) as e:
        ora.floatbits(np.array([1.0, np.inf], dtype=np.float32), [23], None)
    assert e.value.code == ora.ERR_NONFINITE
    bf = (g.view(np.uint32) >> 16).astype(np.uint16)
    mbf = ora.floatbits(bf, [1, 3, 7], None, force_level=2)
    assert np.array_equal(mbf.est, (bf.astype(np.uint32) << 16).view(np.float32).astype(np.float64) * 0
                          + ora.float_compress(bf, 0) + (ora.float_compress(bf, 7) - ora.float_compress(bf, 3)) / mbf.p_sel)


def test_aggregate_dense_hand_example(ora):
    rows = [np.array([1.0, -2.0, 0.0]), np.array([-3.0, -2.0, 0.5]), np.array([0.5, 1.0, 0.25]), np.array([0.5, 0.0, 0.25])]
    out, scale = ora.aggregate_dense(rows, 3)      # M = 4: mean and mean of magnitudes, typed in by hand
    assert out.tolist() == [-0.25, -0.75, 0.25] and scale.tolist() == [1.25, 1.25, 0.25]


# ----------------------------------------------------------------------------------------------
# s-Top-k (Sec. 2.2, App. D)
# ----------------------------------------------------------------------------------------------
def test_stopk_residual_is_the_segment_of_lth_largest_norm(ora):
    rng = np.random.default_rng(44)
    d, s = 103, 10
    g = rng.standard_normal(d).astype(np.float32)
    g[5] = g[50] = 1.25                                              # a tie across the order
    L = -(-d // s)
    order = sorted(range(d), key=lambda i: (-abs(float(g[i])), i))   # sorted vector, ties by lower index
    segs = [order[l * s:(l + 1) * s] for l in range(L)]
    norms = [float(np.sqrt(np.sum(g[seg].astype(np.float64) ** 2))) for seg in segs]
    assert all(norms[i] >= norms[i + 1] for i in range(L - 1))       # so "k segments of largest norm" are the first k
    for l in range(L):
        m = ora.stopk(g, s, None, force_level=l)
        assert sorted(segs[l]) == m.idx.tolist()                     # Sec. 3.2: the residual is the l-th segment
        assert np.allclose(m.delta, norms, rtol=1e-14)
        assert np.allclose(m.p, np.array(norms) / sum(norms), rtol=1e-14)          # Lemma 3.4 / App. D
        assert np.allclose(m.val.astype(np.float64), g[m.idx].astype(np.float64) / m.p_sel, rtol=1e-7)
    # the same thing as Top-k with the uniform schedule
    k = [min(d, s * (l + 1)) for l in range(L)]
    a, b = ora.stopk(g, s, None, seed=1, step=2, worker=3), ora.topk(g, k, None, seed=1, step=2, worker=3)
    assert a.level == b.level and np.array_equal(a.idx, b.idx) and np.array_equal(a.val, b.val)
    # s = 1 recovers Top-k with the unit schedule (importance sampling case): second moment ||g||_1^2
    u = ora.stopk(g[:20], 1, None, force_level=0)
    assert np.isclose(np.sum(u.delta ** 2 / u.p), np.sum(np.abs(g[:20].astype(np.float64))) ** 2, rtol=1e-13)


# ----------------------------------------------------------------------------------------------
# RTN (Sec. 3.2, App. G)
# ----------------------------------------------------------------------------------------------
def test_rtn_grid_values_against_exact_rational_rounding(ora):
    """C^l(v) = clip(delta round(v / delta), -c, c), delta = 2c / (2^r - 1): recomputed in exact rationals.  The oracle
    takes the rounding decision in fp32 (one multiply by the rounded reciprocal), so an entry may land on the other
    neighbouring grid point only when v / delta is within fp32 rounding of a half-integer; elsewhere the grid index
    must be the exact one, and the value must be that index times delta to fp32 accuracy."""
    rng = np.random.default_rng(45)
    g = rng.standard_normal(600).astype(np.float32)
    c = Fraction(float(np.abs(g).max()))
    for li, r in enumerate([1, 2, 4, 8, 16]):
        got = ora.rtn_compress(g, [1, 2, 4, 8, 16], li)
        delta = 2 * c / (2 ** r - 1)
        for i in range(0, 600, 7):
            t = Fraction(float(g[i])) / delta
            k = round(t)                                             # Python rounds halves to even, like the oracle
            exact = max(-c, min(c, k * delta))
            near_half = abs(abs(t - k) - Fraction(1, 2)) < Fraction(1, 2 ** 18) * max(1, abs(t))
            if not near_half:
                assert abs(Fraction(got[i]) - exact) <= abs(exact) * Fraction(1, 2 ** 22) + Fraction(1, 2 ** 140)
        assert np.all(np.abs(got) <= float(c))
    assert np.array_equal(ora.rtn_compress(g, [1, 2, 4, 8, 16], 5), g.astype(np.float64))   # top level = identity
    # r = 1: the grid is {-2c, 0, 2c}, only |v| > c leaves 0: everything rounds to 0 (the tie at |v| = c goes to even)
    assert not ora.rtn_compress(g, [1, 2, 4, 8, 16], 0).any()
    # distortion of a level: half a step, except where clipping acts
    got = ora.rtn_compress(g, [8], 0)
    assert np.all(np.abs(got - g.astype(np.float64)) <= float(c) / 255 * (1 + 1e-6))


def test_rtn_mlmc_estimate(ora):
    rng = np.random.default_rng(46)
    g = (rng.standard_normal(2000) * 10.0 ** rng.uniform(-2, 0, 2000)).astype(np.float32)
    r = [2, 4, 8, 16]
    L = len(r) + 1
    levels = [ora.rtn_compress(g, r, l) for l in range(L)]
    mean, second = np.zeros(g.size), 0.0
    for l in range(L):
        m = ora.rtn(g, r, None, force_level=l)
        res = levels[l] - (levels[l - 1] if l else 0.0)
        assert np.isclose(m.delta[l], np.sqrt(np.sum(res ** 2)), rtol=1e-14)
        assert np.allclose(m.val.astype(np.float64), res / m.p_sel, rtol=1e-7, atol=0)
        assert np.allclose(m.p, m.delta / m.delta.sum(), rtol=1e-15)            # Lemma 3.4
        mean += m.p_sel * (res / m.p_sel)
        second += np.sum(res ** 2) / m.p_sel
    assert np.allclose(mean, g.astype(np.float64), rtol=1e-12, atol=1e-18)      # Lemma 3.2: unbiased for C^L(g) = g
    assert np.isclose(second, m.delta.sum() ** 2, rtol=1e-13)                   # Lemma 3.4: second moment (sum Delta)^2
    f = ora.rtn(g, r, [0.2] * 5, seed=3, step=4, worker=5)
    assert np.allclose(f.p, 0.2) and f.u == ora.uniform(3, 4, 5) and f.c == float(np.abs(g).max())
    z = ora.rtn(np.zeros(10, dtype=np.float32), r, None)
    assert z.level == 0 and not z.val.any() and z.p.tolist() == [1.0, 0, 0, 0, 0]
    for bad in ([2, 2], [4, 2], [17]):
        with pytest.raises(ora.OracleError) as e:
            ora.rtn(g, bad, None)
        assert e.value.code == ora.ERR_SCHEDULE
