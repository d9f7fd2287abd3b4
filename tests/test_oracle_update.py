"""Pins for the oracle's update path against what the paper fixes (Eqs. 5-8, Algorithms 1 and 2,
Sec. 5): closed forms, invariants, brute force on 16-element tensors, replay == stored residual."""
import itertools

import numpy as np
import pytest

from paper_2602_03120_b200 import workloads as wl


def _tensor(qo, codes, bits=4, cols=None, **kw):
    codes = np.asarray(codes, np.int32)
    cols = cols or codes.size
    t = qo.Tensor(bits=bits, rows=codes.size // cols, cols=cols, **kw)
    return t, qo.pack(bits, codes)


def _literal_passes(qo, t, codes, seeds, fit, K, hp, e0=None, replay_only=False):
    """Algorithm 2 as whole-tensor numpy passes, one array statement per line of the listing."""
    tc = t.c()
    J = np.arange(codes.size, dtype=np.uint64) + np.uint64(t.elem_offset)
    W = codes.astype(np.float64)
    e = np.zeros(codes.size) if e0 is None else np.asarray(e0, np.float64).copy()
    N = hp.n_pop
    gens = K if replay_only else K + 1
    for k in range(gens):
        g = np.zeros(codes.size)
        for i in range(N):
            d, _, _ = qo.delta(int(seeds[k, i]), J, hp.sigma)
            g += float(fit[k, i]) * d
        g /= (N * float(np.float32(hp.sigma)))
        u = float(np.float32(hp.lr)) * g + float(np.float32(hp.gamma)) * e
        step = np.sign(u) * np.floor(np.abs(u) + 0.5)
        target = W + step
        if hp.boundary_mode == 0:
            final = np.where((target >= tc.qmin) & (target <= tc.qmax), step, 0.0)
        else:
            final = np.clip(target, tc.qmin, tc.qmax) - W
        e = u - final
        if k == K and not replay_only:
            W = W + final
    return W.astype(np.int32), e


def test_single_member_zero_residual_is_rounded_scaled_noise(qo):
    """N = 1, e = 0: Delta W = Round(alpha * F * delta / sigma) (Eq. 5 into Eqs. 6-7)."""
    n = 4096
    codes = np.zeros(n, np.int32)
    t, w = _tensor(qo, codes, bits=8, cols=64)
    for (sigma, lr, F, gamma) in ((0.5, 1.0, 1.0, 0.9), (1.5, 0.3, -2.0, 0.0), (0.75, 2.0, 0.5, 1.0)):
        hp = qo.HParams(sigma=sigma, lr=lr, gamma=gamma, n_pop=1)
        seeds = np.array([[0xABCDEF]], np.uint64); fit = np.array([[F]], np.float32)
        out = qo.update(t, w, None, seeds, fit, 0, hp)
        d, _, _ = qo.delta(0xABCDEF, np.arange(n, dtype=np.uint64), sigma)
        u = float(np.float32(lr)) * F * d / float(np.float32(sigma))
        want = np.sign(u) * np.floor(np.abs(u) + 0.5)
        assert np.array_equal(out["w_new"], want.astype(np.int32))
        assert np.allclose(out["e_new"], u - want, atol=1e-12)
        assert np.any(want != 0)


def test_ties_round_away_from_zero(qo):
    """|u| = 0.5 crosses the threshold (Sec. 3.2: "|u| >= 0.5")."""
    n = 2048
    t, w = _tensor(qo, np.zeros(n, np.int32), bits=8, cols=64)
    hp = qo.HParams(sigma=0.5, lr=0.25, gamma=1.0, n_pop=1)      # c = 0.5
    seeds = np.array([[42]], np.uint64); fit = np.array([[1.0]], np.float32)
    out = qo.update(t, w, None, seeds, fit, 0, hp)
    d, _, _ = qo.delta(42, np.arange(n, dtype=np.uint64), 0.5)
    assert np.any(d == 1) and np.any(d == -1)
    assert np.all(out["w_new"][d == 1] == 1) and np.all(out["w_new"][d == -1] == -1)
    assert np.all(out["band"][np.abs(d) == 1] == 0.0)


def test_zero_fitness_leaves_weights_and_decays_residual(qo):
    n = 1024
    rng = np.random.default_rng(3)
    codes = rng.integers(-8, 8, n).astype(np.int32)
    t, w = _tensor(qo, codes, cols=64)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=4)
    e_in = rng.uniform(-0.5, 0.5, n).astype(np.float32)
    out = qo.update(t, w, None, wl.draw_seeds(1, 4), np.zeros((1, 4), np.float32), 0, hp, residual_in=e_in)
    assert np.array_equal(out["w_new"], codes)
    assert np.allclose(out["e_new"], float(np.float32(0.9)) * e_in.astype(np.float64), atol=1e-12)


def test_residual_stays_within_half_a_step_unless_gated(qo):
    """Sec. 5: |e| <= Delta/2 wherever the step was applied; a gated step keeps all of u."""
    n = 1 << 14
    codes = np.random.default_rng(1).integers(-8, 8, n).astype(np.int32)
    t, w = _tensor(qo, codes, cols=128)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    K = 6
    seeds, fit = wl.draw_seeds(K + 1, 8), wl.draw_fitness(K + 1, 8)
    out = qo.update(t, w, None, seeds, fit, K, hp)
    free = out["gate_final"] == 0
    assert np.all(np.abs(out["e_new"][free]) <= 0.5 + 1e-12)
    assert np.any(~free)
    assert np.all(out["w_new"][~free] == codes[~free])
    assert np.all(np.abs(out["e_new"][~free]) >= 0.5 - 1e-12)
    assert out["w_new"].min() >= -8 and out["w_new"].max() <= 7


@pytest.mark.parametrize("mode", [0, 1])
def test_brute_force_sixteen_element_tensor(qo, mode):
    """All 16 INT4 codes, N <= 2, K <= 2, fitness in {-1, 0, 1}: every table, both boundary modes,
    element-wise oracle vs the listing written as whole-tensor passes."""
    codes = np.arange(-8, 8, dtype=np.int32)
    t, w = _tensor(qo, codes, cols=16, elem_offset=64)
    checked = 0
    for N, K in ((1, 0), (1, 2), (2, 1), (2, 2)):
        seeds = wl.draw_seeds(K + 1, N, stream=10 * N + K)
        hp = qo.HParams(sigma=1.5, lr=1.0, gamma=0.9, n_pop=N, boundary_mode=mode)
        for table in itertools.product((-1.0, 0.0, 1.0), repeat=N * (K + 1)):
            fit = np.array(table, np.float32).reshape(K + 1, N)
            out = qo.update(t, w, None, seeds, fit, K, hp)
            W, e = _literal_passes(qo, t, codes, seeds, fit, K, hp)
            assert np.array_equal(out["w_new"], W)
            assert np.allclose(out["e_new"], e, atol=1e-12)
            checked += 1
    assert checked == 3 + 27 + 81 + 729


def test_replay_matches_explicit_passes_and_replay_entry(qo):
    n = 4096
    codes = np.random.default_rng(8).integers(-8, 8, n).astype(np.int32)
    t, w = _tensor(qo, codes, cols=256, elem_offset=1 << 20)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    K = 5
    seeds, fit = wl.draw_seeds(K + 1, 8, stream=2), wl.draw_fitness(K + 1, 8, stream=2)
    W, e = _literal_passes(qo, t, codes, seeds, fit, K, hp)
    out = qo.update(t, w, None, seeds, fit, K, hp)
    assert np.array_equal(out["w_new"], W) and np.allclose(out["e_new"], e, atol=1e-12)
    _, e_hist = _literal_passes(qo, t, codes, seeds[:K], fit[:K], K, hp, replay_only=True)
    rep = qo.replay_residual(t, w, None, seeds[:K], fit[:K], K, hp)
    assert np.allclose(rep["e"], e_hist, atol=1e-12)
    # the stateless update is one stored-residual step started from the replayed residual
    one = qo.update(t, w, None, seeds[K:], fit[K:], 0, hp, residual_in=rep["e"].astype(np.float32))
    far = out["band"] > 1e-6
    assert np.array_equal(one["w_new"][far], out["w_new"][far])


def test_replayed_residual_equals_stored_residual_on_true_trajectory(qo):
    """Algorithm 1 run step by step with the residual kept in memory, then Algorithm 2's history loop
    over the same generations: identical where the gate cannot fire (Sec. 3.3)."""
    n = 2048
    codes = np.random.default_rng(4).integers(-64, 64, n).astype(np.int32)
    t, w = _tensor(qo, codes, bits=8, cols=128)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    T = 8
    seeds, fit = wl.draw_seeds(T, 8, stream=3), wl.draw_fitness(T, 8, stream=3)
    e = np.zeros(n, np.float64); cur = w.copy()
    for s in range(T):
        out = qo.update(t, cur, None, seeds[s:s + 1], fit[s:s + 1], 0, hp, residual_in=e.astype(np.float32))
        # keep the residual in double across steps: feed it back through a float64-exact path
        e_prev = e
        out64 = _literal_passes(qo, t, qo.unpack(8, cur, n), seeds[s:s + 1], fit[s:s + 1], 0, hp, e0=e_prev)
        cur = qo.pack(8, out64[0]); e = out64[1]
        far = out["band"] > 1e-6
        assert np.array_equal(out["w_new"][far], out64[0][far])
    rep = qo.replay_residual(t, cur, None, seeds, fit, T, hp)
    assert np.all(rep["gate_replay"] == 0)
    assert np.allclose(rep["e"], e, atol=1e-12)
    assert np.any(qo.unpack(8, cur, n) != codes)
    # truncated window: difference bounded by gamma^K times the residual bound (Sec. 3.3)
    Kt = 5
    rep_t = qo.replay_residual(t, cur, None, seeds[T - Kt:], fit[T - Kt:], Kt, hp)
    diff = np.abs(rep_t["e"] - e)
    settled = diff <= 0.9 ** Kt * 0.5 + 1e-12
    # where the forgotten residual flips no rounding decision the difference is exactly gamma^K e_{T-K};
    # a flipped decision moves the residual by a whole step, which then decays by gamma per generation
    assert settled.mean() > 0.5
    assert diff.max() <= 0.9 ** Kt * 0.5 + sum(0.9 ** s for s in range(Kt)) + 1e-12


def test_temporal_equivalence_gamma_one_no_gate(qo):
    """Sec. 5: with gamma = 1 and no gating, W_T + e_T = W_0 + sum_t alpha * g_t exactly."""
    n = 1024
    codes = np.zeros(n, np.int32)
    t, w = _tensor(qo, codes, bits=8, cols=64)
    hp = qo.HParams(sigma=0.5, lr=0.7, gamma=1.0, n_pop=4)
    T = 10
    seeds, fit = wl.draw_seeds(T, 4, stream=5), wl.draw_fitness(T, 4, stream=5)
    J = np.arange(n, dtype=np.uint64)
    ideal = np.zeros(n)
    for s in range(T):
        g = sum(float(fit[s, i]) * qo.delta(int(seeds[s, i]), J, 0.5)[0] for i in range(4)) / (4 * 0.5)
        ideal += float(np.float32(0.7)) * g
    W, e = codes.astype(np.float64), np.zeros(n)
    for s in range(T):
        Wn, e = _literal_passes(qo, t, W.astype(np.int32), seeds[s:s + 1], fit[s:s + 1], 0, hp, e0=e)
        W = Wn.astype(np.float64)
    assert np.abs(W + e - ideal).max() < 1e-9
    assert np.abs(e).max() <= 0.5 + 1e-12
    # the same final state from the stateless path with the whole history in the window
    out = qo.update(t, w, None, seeds, fit, T - 1, hp)
    far = out["band"] > 1e-9
    # replay gates/rounds identically here (no gate fires; W_t enters only through the gate)
    assert np.allclose((out["e_new"])[far], e[far], atol=1e-9)


def test_stagnation_without_residual_and_accumulation_with_it(qo):
    """Sec. 3.2 / Sec. 5: |alpha g| < 1/2 never moves a weight without error feedback (gamma = 0),
    while the carried residual fires a step once the accumulated signal crosses 1/2."""
    n = 512
    t, w = _tensor(qo, np.zeros(n, np.int32), bits=8, cols=64)
    seeds = wl.draw_seeds(1, 1, stream=9)
    fit = np.ones((1, 1), np.float32)
    J = np.arange(n, dtype=np.uint64)
    d = qo.delta(int(seeds[0, 0]), J, 0.5)[0]
    lr = 0.1                                           # c = 0.2: a unit delta gives u = 0.2
    pick = d == 1
    assert pick.sum() > 10
    # no feedback: the same generation applied 5 times never moves the weight
    hp0 = qo.HParams(sigma=0.5, lr=lr, gamma=0.0, n_pop=1)
    cur = w.copy()
    for _ in range(5):
        out = qo.update(t, cur, None, seeds, fit, 0, hp0, residual_in=np.zeros(n, np.float32))
        cur = qo.pack(8, out["w_new"])
    assert np.all(qo.unpack(8, cur, n)[pick] == 0)
    # with feedback (gamma = 1): u = 0.2, 0.4, 0.6 -> fires on the third step, residual -0.4
    hp1 = qo.HParams(sigma=0.5, lr=lr, gamma=1.0, n_pop=1)
    cur, e, hist = w.copy(), np.zeros(n, np.float32), []
    for _ in range(3):
        out = qo.update(t, cur, None, seeds, fit, 0, hp1, residual_in=e)
        cur = qo.pack(8, out["w_new"]); e = out["e_new"].astype(np.float32)
        hist.append(out["w_new"][pick].copy())
    assert np.all(hist[0] == 0) and np.all(hist[1] == 0) and np.all(hist[2] == 1)
    assert np.allclose(e[pick], -0.4, atol=1e-6)


def test_result_independent_of_tensor_split_and_threads(qo):
    rows, cols = 8, 128
    codes = np.random.default_rng(6).integers(-8, 8, rows * cols).astype(np.int32)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=4)
    K = 2
    seeds, fit = wl.draw_seeds(K + 1, 4, stream=7), wl.draw_fitness(K + 1, 4, stream=7)
    whole, ww = _tensor(qo, codes, cols=cols, elem_offset=4096)
    full = qo.update(whole, ww, None, seeds, fit, K, hp, nthreads=1)
    full8 = qo.update(whole, ww, None, seeds, fit, K, hp, nthreads=8)
    assert np.array_equal(full["w_new"], full8["w_new"]) and np.array_equal(full["e_new"], full8["e_new"])
    half = rows // 2 * cols
    top, wt = _tensor(qo, codes[:half], cols=cols, elem_offset=4096)
    bot, wb = _tensor(qo, codes[half:], cols=cols, elem_offset=4096 + half)
    a = qo.update(top, wt, None, seeds, fit, K, hp)
    b = qo.update(bot, wb, None, seeds, fit, K, hp)
    assert np.array_equal(np.concatenate([a["w_new"], b["w_new"]]), full["w_new"])
    idx = np.array([5, 77, 1000], np.int64)
    part = qo.update(whole, ww, None, seeds, fit, K, hp, idx=idx)
    assert np.array_equal(part["w_new"], full["w_new"][idx])
    # a different offset is a different noise stream
    other, wo = _tensor(qo, codes, cols=cols, elem_offset=8192)
    assert not np.array_equal(qo.update(other, wo, None, seeds, fit, K, hp)["e_new"], full["e_new"])


def test_perturb_is_gated_delta_and_consistent_with_update(qo):
    """Algorithm 1: W' = Gate(W + delta_i); the delta implied by perturb is the one the update sums."""
    rows, cols = 16, 128
    n = rows * cols
    codes = np.random.default_rng(2).integers(-8, 8, n).astype(np.int32)
    t, w = _tensor(qo, codes, cols=cols, elem_offset=96)
    hp = qo.HParams(sigma=1.0, lr=1.0, gamma=0.9, n_pop=1)
    seed = 0x5EED5EED5EED
    wp = qo.perturb(t, w, None, seed, hp)
    d = qo.delta(seed, np.arange(n, dtype=np.uint64) + np.uint64(96), 1.0)[0]
    inside = (codes + d >= -8) & (codes + d <= 7)
    assert np.array_equal(wp, np.where(inside, codes + d, codes))
    assert np.any(~inside) and np.any(d != 0)
    hp_c = qo.HParams(sigma=1.0, lr=1.0, gamma=0.9, n_pop=1, boundary_mode=1)
    assert np.array_equal(qo.perturb(t, w, None, seed, hp_c), np.clip(codes + d, -8, 7))
    # one-member update with F = sigma (so c * F = 1) steps by exactly delta where not gated
    up = qo.update(t, w, None, np.array([[seed]], np.uint64), np.array([[1.0]], np.float32), 0, hp)
    assert np.array_equal(up["w_new"], wp)


def test_weight_unit_sigma_uses_group_scale(qo):
    """sigma given in weight units: the grid-unit sigma of a group is sigma / scale (App. A grid)."""
    rows, cols, group = 4, 256, 128
    n = rows * cols
    codes = np.zeros(n, np.int32)
    t, w = _tensor(qo, codes, bits=8, cols=cols, group_size=group)
    scales = np.array([0.01, 0.02, 0.04, 0.005, 0.01, 0.02, 0.04, 0.005], np.float16)
    hp = qo.HParams(sigma=0.02, lr=1.0, gamma=0.9, n_pop=1, sigma_unit=1)
    wp = qo.perturb(t, w, scales, 123, hp)
    J = np.arange(n, dtype=np.uint64)
    for g in range(rows * cols // group):
        seff = float(np.float32(0.02) / np.float32(scales[g]))
        sl = slice(g * group, (g + 1) * group)
        assert np.array_equal(wp[sl], qo.delta(123, J[sl], seff)[0])
    # per-row scales (group_size 0)
    t2, _ = _tensor(qo, codes, bits=8, cols=cols, group_size=0)
    wp2 = qo.perturb(t2, w, scales[:rows], 123, hp)
    for r in range(rows):
        seff = float(np.float32(0.02) / np.float32(scales[r]))
        sl = slice(r * cols, (r + 1) * cols)
        assert np.array_equal(wp2[sl], qo.delta(123, J[sl], seff)[0])


def test_history_buffer_is_twelve_bytes_per_member(qo):
    """App. D: the optimizer state at K = 50, N = 50 is about 29.7 KB (u64 seed + f32 reward each)."""
    seeds, fit = wl.draw_seeds(50, 50), wl.draw_fitness(50, 50)
    assert seeds.nbytes + fit.nbytes == 30000
    assert abs(30000 / 1024 - 29.7) / 29.7 < 0.02
