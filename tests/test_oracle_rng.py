"""Pins for the oracle's noise generator: Philox known answers, Box-Muller against libm,
stochastic rounding (Eq. 3) against its definition and its expectation."""
import os
from fractions import Fraction

import numpy as np
from scipy import stats

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers(qo):
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        out = qo.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


def test_philox_counter_and_key_are_not_interchangeable(qo):
    a = qo.philox4x32_10([1, 0, 0, 0], [0, 0])
    b = qo.philox4x32_10([0, 1, 0, 0], [0, 0])
    c = qo.philox4x32_10([0, 0, 0, 0], [1, 0])
    d = qo.philox4x32_10([0, 0, 0, 0], [0, 1])
    outs = [tuple(int(v) for v in x) for x in (a, b, c, d)]
    assert len(set(outs)) == 4


def _all24():
    return (np.arange(1 << 24, dtype=np.uint64) << 8).astype(np.uint32)


def test_bm24_radius_exhaustive_against_libm(qo):
    r0 = _all24()
    R, _, _ = qo.bm24(r0, r0)
    n = (r0 >> 8).astype(np.float64) + 1.0
    ref = np.sqrt(-2.0 * np.log(n / 2.0 ** 24))
    err = np.abs(R.astype(np.float64) - ref)
    assert err.max() <= 5e-7
    assert (err / (1.0 + ref)).max() <= 1.5e-7
    assert R[-1] == 0.0 and R.min() == 0.0                     # u1 = 1 -> radius 0
    assert abs(float(R[0]) - np.sqrt(48 * np.log(2.0))) < 1e-6   # u1 = 2^-24 -> sqrt(48 ln 2)


def test_bm24_cos_sin_exhaustive_against_libm(qo):
    r1 = _all24()
    _, c, s = qo.bm24(r1, r1)
    th = 2.0 * np.pi * (r1 >> 8).astype(np.float64) / 2.0 ** 24
    assert np.abs(c - np.cos(th)).max() <= 1.5e-7
    assert np.abs(s - np.sin(th)).max() <= 1.5e-7
    assert np.abs(c.astype(np.float64) ** 2 + s.astype(np.float64) ** 2 - 1.0).max() <= 4e-7
    # exact values on the axes
    for k, (cc, ss) in {0: (1, 0), 1 << 22: (0, 1), 1 << 23: (-1, 0), 3 << 22: (0, -1)}.items():
        assert c[k] == cc and s[k] == ss


def test_noise_is_standard_normal(qo):
    n = 2_000_000
    J = np.arange(n, dtype=np.uint64)
    _, x, _ = qo.delta(0x1234_5678_9ABC_DEF0, J, 1.0, tier=qo.TIER_SPEC)
    assert abs(x.mean()) < 4 / np.sqrt(n)
    assert abs(x.var() - 1.0) < 4 * np.sqrt(2.0 / n)
    assert abs(stats.skew(x)) < 4 * np.sqrt(6.0 / n)
    assert abs(stats.kurtosis(x)) < 4 * np.sqrt(24.0 / n)
    assert stats.kstest(x[:500_000], "norm").pvalue > 1e-3
    # even / odd members of a pair come from cos / sin of the same angle: uncorrelated
    assert abs(np.corrcoef(x[0::2], x[1::2])[0, 1]) < 4 / np.sqrt(n / 2)


def test_delta_wiring_matches_manual_composition(qo):
    """delta(seed, J) == Eq. 3 applied to Box-Muller of Philox(key=seed halves, ctr=(lo p, hi p, 0, 0))."""
    seed = 0xDEADBEEF_01234567
    J = np.array([0, 1, 2, 3, 1000, 1001, (1 << 33) + 6, (1 << 33) + 7, (1 << 40) + 123], dtype=np.uint64)
    sig = 1.7
    d, x, _ = qo.delta(seed, J, sig, tier=qo.TIER_SPEC)
    for i, j in enumerate(J):
        p = int(j) >> 1
        r = qo.philox4x32_10([p & 0xffffffff, p >> 32, 0, 0], [seed & 0xffffffff, seed >> 32])
        R, c, s = qo.bm24(r[0:1], r[1:2])
        trig = s[0] if (int(j) & 1) else c[0]
        xx = np.float32(np.float32(sig) * R[0]) * trig
        assert np.float32(xx) == np.float32(x[i])
        # Eq. 3 decided exactly: 24-bit integer uniform against the exact fractional part of the fp32 x
        xq = Fraction(float(np.float32(xx)))
        fl = xq.numerator // xq.denominator
        want = fl + (1 if Fraction(int(r[3 if (int(j) & 1) else 2]) >> 8, 1 << 24) < xq - fl else 0)
        assert d[i] == max(-8, min(7, want))


def test_plain_and_spec_tiers_agree_except_near_decisions(qo):
    n = 4_000_000
    J = np.arange(n, dtype=np.uint64) + (1 << 35)
    ds, xs, _ = qo.delta(77, J, 0.5, tier=qo.TIER_SPEC)
    dp, xp, near = qo.delta(77, J, 0.5, tier=qo.TIER_PLAIN, tau=1e-5)
    assert np.abs(xs - xp).max() < 2e-6
    differ = ds != dp
    assert not np.any(differ & (near == 0))
    assert near.mean() < 1e-4


def test_stochastic_rounding_unbiased_and_two_valued(qo):
    rng = np.random.default_rng(5)
    words = rng.integers(0, 1 << 32, size=200_000, dtype=np.uint64)
    for x in (-2.75, -0.3, 0.0, 0.125, 0.5, 1.9, 3.0):
        d = np.array([qo.stochastic_round(x, int(w)) for w in words[:50_000]])
        fl = int(np.floor(x))
        assert set(np.unique(d)) <= {fl, fl + 1}
        frac = x - fl
        assert abs(d.mean() - x) < 4 * np.sqrt(max(frac * (1 - frac), 1e-12) / d.size) + 1e-12
        if frac == 0:
            assert np.all(d == fl)
    # 4-bit range of the perturbation tensor
    assert qo.stochastic_round(9.5, 0) == 7 and qo.stochastic_round(-11.2, 0xffffffff) == -8


def test_bernoulli_threshold_is_the_exact_fraction(qo):
    """Eq. 3: b ~ Bernoulli(x - floor(x)).  For x in (-1/2, 0) the difference x - floor(x) does not fit
    fp32; the decision must use its exact value, so of the 2^24 equally likely uniforms exactly
    ceil((x - floor(x)) * 2^24) give b = 1."""
    x = -(2.0 ** -3 + 3 * 2.0 ** -26)                 # exact in fp32; (x + 1) * 2^24 = 14680063.25
    assert float(np.float32(x)) == x
    assert qo.stochastic_round(x, 14680063 << 8) == 0     # v = 14680063 / 2^24 < x + 1  -> b = 1
    assert qo.stochastic_round(x, 14680064 << 8) == -1    # v = 14680064 / 2^24 > x + 1  -> b = 0
    assert qo.stochastic_round(x, (14680063 << 8) | 0xff) == 0   # the low 8 bits of the word are unused
    # integer x: fraction 0, b = 0 for every uniform, including v = 0
    assert qo.stochastic_round(2.0, 0) == 2 and qo.stochastic_round(-3.0, 0) == -3
    # smallest positive fraction: only v = 0 gives b = 1
    assert qo.stochastic_round(2.0 ** -30, 0) == 1 and qo.stochastic_round(2.0 ** -30, 1 << 8) == 0


def test_expected_delta_equals_sigma_eps(qo):
    """E[delta | eps] = sigma * eps (Eq. 3 is unbiased): averaged over many elements the
    discrete perturbation tracks the continuous one."""
    n = 2_000_000
    J = np.arange(n, dtype=np.uint64)
    d, x, _ = qo.delta(99, J, 0.5, tier=qo.TIER_SPEC)
    resid = d - x
    assert abs(resid.mean()) < 4 * 0.5 / np.sqrt(n)
    assert np.all((resid > -1.0) & (resid <= 1.0))
    assert abs(np.corrcoef(resid, x)[0, 1]) < 4 / np.sqrt(n)


def test_pair_deltas_is_delta_on_the_words_philox_produces(qo):
    """pair_deltas (Box-Muller + Eq. 3 on given words) composed with Philox is delta(seed, J); and on its own
    it follows Eq. 3 when the uniform word is moved across the exact threshold."""
    seed = 0x0BADC0DE_CAFEF00D
    pairs = np.array([0, 1, 77, (1 << 32) + 5, (1 << 39) + 1], dtype=np.uint64)
    words = np.stack([qo.philox4x32_10([int(p) & 0xffffffff, int(p) >> 32, 0, 0], [seed & 0xffffffff, seed >> 32])
                      for p in pairs])
    for sig, dmin in ((0.5, -8), (1.7, -8), (3.0, -7)):
        de, do = qo.pair_deltas(words[:, 0], words[:, 1], words[:, 2], words[:, 3], sig, dmin)
        J = np.stack([2 * pairs, 2 * pairs + 1], axis=1).reshape(-1)
        want = qo.delta(seed, J, sig, dmin=dmin)[0].reshape(-1, 2)
        assert np.array_equal(de, want[:, 0]) and np.array_equal(do, want[:, 1])
    # threshold: x = sigma * R * cos with the uniform just below / at the exact fraction
    r0, r1 = words[:1, 0], words[:1, 1]
    R, c, _ = qo.bm24(r0, r1)
    x = Fraction(float(np.float32(np.float32(0.5) * R[0]) * c[0]))
    fl = x.numerator // x.denominator
    k = -((-(x - fl) * (1 << 24)).__floor__())          # ceil(frac * 2^24): uniforms 0 .. k-1 give b = 1
    below = np.array([(k - 1) << 8], np.uint32); at = np.array([k << 8], np.uint32)
    assert qo.pair_deltas(r0, r1, below, below, 0.5)[0][0] == fl + 1
    assert qo.pair_deltas(r0, r1, at, at, 0.5)[0][0] == fl
