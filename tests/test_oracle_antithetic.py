"""Pins for antithetic perturbation pairs (App. A: "N antithetic perturbation pairs per generation") in the
oracle: a pair is one seed and the two members W + delta, W - delta; Eq. 5 sums over all N members."""
import numpy as np

from paper_2602_03120_b200 import workloads as wl


def _tensor(qo, codes, bits=8, cols=None, **kw):
    codes = np.asarray(codes, np.int32)
    cols = cols or codes.size
    return qo.Tensor(bits=bits, rows=codes.size // cols, cols=cols, **kw), qo.pack(bits, codes)


def _explicit_members(qo, t, codes, seeds, fit, K, hp):
    """Algorithm 2 with every one of the N members written out: member 2j uses +delta_j, member 2j+1 -delta_j."""
    tc = t.c()
    J = np.arange(codes.size, dtype=np.uint64) + np.uint64(t.elem_offset)
    W = codes.astype(np.float64)
    e = np.zeros(codes.size)
    N = hp.n_pop
    for k in range(K + 1):
        members = []
        for j in range(N // 2):
            d, _, _ = qo.delta(int(seeds[k, j]), J, hp.sigma, dmin=-7)
            members += [d.astype(np.float64), -d.astype(np.float64)]
        g = sum(float(fit[k, i]) * members[i] for i in range(N)) / (N * float(np.float32(hp.sigma)))
        u = float(np.float32(hp.lr)) * g + float(np.float32(hp.gamma)) * e
        step = np.sign(u) * np.floor(np.abs(u) + 0.5)
        target = W + step
        final = np.where((target >= tc.qmin) & (target <= tc.qmax), step, 0.0)
        e = u - final
        if k == K:
            W = W + final
    return W.astype(np.int32), e


def test_pairs_equal_the_sum_over_all_explicit_members(qo):
    rng = np.random.default_rng(11)
    codes = rng.integers(-8, 8, 2048)
    t, w = _tensor(qo, codes, bits=4, cols=64, elem_offset=64)
    N, K = 6, 3
    seeds = wl.draw_seeds(K + 1, N // 2, stream=41)
    fit = wl.draw_fitness(K + 1, N, stream=41)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N, antithetic=1)
    out = qo.update(t, w, None, seeds, fit, K, hp)
    W, e = _explicit_members(qo, t, codes, seeds, fit, K, hp)
    far = out["band"] > 1e-9
    assert np.array_equal(out["w_new"][far], W[far]) and far.mean() > 0.999
    assert np.abs(out["e_new"] - e)[far].max() < 1e-9
    rr = qo.replay_residual(t, w, None, seeds[:K], fit[:K], K, hp)
    assert rr["e"].shape == (2048,)


def test_pairs_reduce_to_half_the_seeds_with_fitness_differences(qo):
    """F+ * delta + F- * (-delta) = (F+ - F-) * delta: an antithetic population of N equals N / 2 plain
    members with fitness F+ - F- at half the learning rate (c = alpha / (N sigma))."""
    codes = np.zeros(1024, np.int32)
    t, w = _tensor(qo, codes, bits=8, cols=64)
    N, K = 8, 2
    seeds = wl.draw_seeds(K + 1, N // 2, stream=42)
    fit = (np.random.default_rng(3).integers(-8, 9, size=(K + 1, N)) / 8.0).astype(np.float32)   # differences exact
    anti = qo.update(t, w, None, seeds, fit, K, qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N, antithetic=1))
    diff = (fit[:, 0::2] - fit[:, 1::2]).astype(np.float32)
    plain = qo.update(t, w, None, seeds, diff, K, qo.HParams(sigma=0.5, lr=0.5, gamma=0.9, n_pop=N // 2))
    assert np.array_equal(anti["w_new"], plain["w_new"])
    assert np.abs(anti["e_new"] - plain["e_new"]).max() < 1e-12
    assert np.any(anti["w_new"] != 0)


def test_equal_fitness_within_every_pair_gives_no_update(qo):
    codes = np.random.default_rng(5).integers(-100, 100, 512)
    t, w = _tensor(qo, codes, bits=8, cols=64)
    fit = np.repeat(wl.draw_fitness(3, 4, stream=43), 2, axis=1)      # F+ == F-
    out = qo.update(t, w, None, wl.draw_seeds(3, 4, stream=43), fit, 2, qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=8, antithetic=1))
    assert np.array_equal(out["w_new"], codes) and np.all(out["e_new"] == 0.0)


def test_the_two_members_of_a_pair_are_mirror_images(qo):
    codes = np.zeros(4096, np.int32)
    t, w = _tensor(qo, codes, bits=8, cols=64)
    for sigma in (0.5, 3.0):                                              # 3.0 reaches the 4-bit limit
        hp = qo.HParams(sigma=sigma, lr=1.0, gamma=0.9, n_pop=2, antithetic=1)
        plus = qo.perturb(t, w, None, 777, hp, sign=1)
        minus = qo.perturb(t, w, None, 777, hp, sign=-1)
        assert np.array_equal(plus, -minus)
        assert plus.min() >= -7 and plus.max() <= 7
        d, _, _ = qo.delta(777, np.arange(4096, dtype=np.uint64), sigma, dmin=-7)
        assert np.array_equal(plus, d)
    assert plus.min() == -7 and plus.max() == 7
    # the gate acts on each member separately
    edge, we = _tensor(qo, np.full(64, 127, np.int32), bits=8, cols=64)
    hp = qo.HParams(sigma=1.0, lr=1.0, gamma=0.9, n_pop=2, antithetic=1)
    p, m = qo.perturb(edge, we, None, 5, hp, sign=1), qo.perturb(edge, we, None, 5, hp, sign=-1)
    d, _, _ = qo.delta(5, np.arange(64, dtype=np.uint64), 1.0, dmin=-7)
    assert np.array_equal(p, np.where(d > 0, 127, 127 + d)) and np.array_equal(m, np.where(d < 0, 127, 127 - d))


def test_odd_population_is_rejected(qo):
    import pytest
    t, w = _tensor(qo, np.zeros(64, np.int32), bits=8, cols=64)
    with pytest.raises(ValueError):
        qo.update(t, w, None, wl.draw_seeds(1, 1), np.zeros((1, 3), np.float32), 0,
                  qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=3, antithetic=1))
