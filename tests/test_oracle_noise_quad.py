"""Pins for the second bit allocation of the noise contract (noise_mode = 1): one Philox call per four
elements, two Box-Muller pairs from the top 24 bits of its words, Bernoulli uniforms from their low bytes."""
from fractions import Fraction

import numpy as np
from scipy import stats

from paper_2602_03120_b200 import workloads as wl


def test_wiring_matches_manual_composition(qo):
    seed = 0x0123456789ABCDEF
    J = np.array([0, 1, 2, 3, 4, 5, 6, 7, 1002, 1003, (1 << 34) + 8, (1 << 34) + 11, (1 << 41) + 5], dtype=np.uint64)
    sig = 1.3
    d, x, _ = qo.delta(seed, J, sig, noise_mode=1)
    for i, j in enumerate(int(v) for v in J):
        q, h = j >> 2, j & 3
        r = qo.philox4x32_10([q & 0xffffffff, q >> 32, 0, 0], [seed & 0xffffffff, seed >> 32])
        R, c, s = qo.bm24(r[(h & 2):(h & 2) + 1], r[(h & 2) + 1:(h & 2) + 2])
        xx = np.float32(np.float32(sig) * R[0]) * (s[0] if h & 1 else c[0])
        assert np.float32(xx) == np.float32(x[i])
        xq = Fraction(float(np.float32(xx)))
        fl = xq.numerator // xq.denominator
        v = Fraction(2 * (int(r[h]) & 0xff) + 1, 512)
        assert d[i] == max(-8, min(7, fl + (1 if v < xq - fl else 0)))


def test_bernoulli_probability_is_the_fraction_to_the_nearest_256th(qo):
    for x in (-2.75, -0.3, 0.0, 0.126, 0.5, 1.9, 3.0, 0.001, 0.999, -0.0019):
        fl = int(np.floor(np.float32(x)))
        frac = float(np.float32(x)) - fl
        ones = sum(qo.stochastic_round_byte(x, b) - fl for b in range(256))
        assert all(qo.stochastic_round_byte(x, b) in (fl, fl + 1) for b in range(256))
        assert abs(ones / 256.0 - frac) <= 1.0 / 512 + 1e-12
        assert ones == int(np.ceil(frac * 256 - 0.5))           # number of v = (b + 1/2)/256 below frac
    assert qo.stochastic_round_byte(2.0, 0) == 2                # integer x: never rounds up


def test_noise_is_standard_normal_and_the_four_elements_of_a_call_are_uncorrelated(qo):
    n = 2_000_000
    J = np.arange(n, dtype=np.uint64) + (1 << 36)
    d, x, _ = qo.delta(0xFEEDFACE12345678, J, 1.0, noise_mode=1)
    assert abs(x.mean()) < 4 / np.sqrt(n) and abs(x.var() - 1.0) < 4 * np.sqrt(2.0 / n)
    assert abs(stats.skew(x)) < 4 * np.sqrt(6.0 / n) and abs(stats.kurtosis(x)) < 4 * np.sqrt(24.0 / n)
    assert stats.kstest(x[:500_000], "norm").pvalue > 1e-3
    quad = x.reshape(-1, 4)
    cc = np.corrcoef(quad.T)
    assert np.abs(cc - np.eye(4)).max() < 4 / np.sqrt(n / 4)
    # the rounding error does not track the noise: the Bernoulli byte is independent of the Gaussian bits
    resid = d - x
    assert np.all((resid > -1.0) & (resid <= 1.0))
    assert abs(resid.mean()) < 4 * 0.5 / np.sqrt(n) + 1e-4
    assert abs(np.corrcoef(resid, x)[0, 1]) < 4 / np.sqrt(n)


def test_modes_draw_different_streams_and_tiers_agree(qo):
    J = np.arange(200_000, dtype=np.uint64)
    d0, x0, _ = qo.delta(5, J, 0.5, noise_mode=0)
    d1, x1, _ = qo.delta(5, J, 0.5, noise_mode=1)
    assert np.array_equal(x0[:2], x1[:2]) and not np.array_equal(x0[:64], x1[:64])   # same first pair, then they part
    dp, xp, near = qo.delta(5, J, 0.5, tier=qo.TIER_PLAIN, tau=1e-5, noise_mode=1)
    assert np.abs(x1 - xp).max() < 2e-6
    assert not np.any((d1 != dp) & (near == 0))


def test_update_with_quad_noise_equals_whole_tensor_passes(qo):
    codes = np.random.default_rng(8).integers(-8, 8, 1024).astype(np.int32)
    t = qo.Tensor(bits=4, rows=16, cols=64, elem_offset=96)
    w = qo.pack(4, codes)
    N, K = 4, 2
    seeds, fit = wl.draw_seeds(K + 1, N, stream=90), wl.draw_fitness(K + 1, N, stream=90)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N, noise_mode=1)
    out = qo.update(t, w, None, seeds, fit, K, hp)
    J = np.arange(1024, dtype=np.uint64) + np.uint64(96)
    W, e = codes.astype(np.float64), np.zeros(1024)
    for k in range(K + 1):
        g = sum(float(fit[k, i]) * qo.delta(int(seeds[k, i]), J, 0.5, noise_mode=1)[0] for i in range(N)) / (N * 0.5)
        u = g + float(np.float32(0.9)) * e
        step = np.sign(u) * np.floor(np.abs(u) + 0.5)
        final = np.where((W + step >= -8) & (W + step <= 7), step, 0.0)
        e = u - final
    far = out["band"] > 1e-9
    assert np.array_equal(out["w_new"][far], (W + final).astype(np.int32)[far])
    assert np.abs(out["e_new"] - e)[far].max() < 1e-9
    plain = qo.update(t, w, None, seeds, fit, K, qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N))
    assert not np.array_equal(plain["w_new"], out["w_new"])
    p1 = qo.perturb(t, w, None, int(seeds[0, 0]), hp)
    d = qo.delta(int(seeds[0, 0]), J, 0.5, noise_mode=1)[0]
    assert np.array_equal(p1, np.where((codes + d >= -8) & (codes + d <= 7), codes + d, codes))
