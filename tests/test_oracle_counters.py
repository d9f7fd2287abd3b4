"""Pins for the oracle's boundary bookkeeping (Algorithm 2, the two Gate(...) lines; Sec. 3.3): the
counters gate_final / gate_replay / attempted and the per-generation record of blocked steps, worked
out from the delta values alone, and the replay-versus-stored gate-mismatch count on a true
trajectory whose gate does fire."""
import numpy as np
import pytest

from paper_2602_03120_b200 import workloads as wl
from stored_trajectory import stored_trajectory


def _tensor(qo, codes, bits=4, cols=None, **kw):
    codes = np.asarray(codes, np.int32)
    cols = cols or codes.size
    t = qo.Tensor(bits=bits, rows=codes.size // cols, cols=cols, **kw)
    return t, qo.pack(bits, codes)


@pytest.mark.parametrize("mode", [0, 1])
def test_counters_from_the_delta_values_without_carry(qo, mode):
    """N = 1, sigma = lr (so alpha / (N sigma) = 1), gamma = 0, fitness +-1: generation k's rounded
    step is exactly F_k * delta_k, nothing is carried, and every counter follows from the integer
    deltas: a step is blocked (gate) or shortened (clamp) exactly when W + F_k delta_k leaves the
    range; history generations count into gate_replay, the last one into gate_final / attempted."""
    reps, K = 6, 3
    codes = np.tile(np.arange(-8, 8, dtype=np.int32), reps)
    n = codes.size
    t, w = _tensor(qo, codes, cols=32, elem_offset=4096)
    hp = qo.HParams(sigma=1.5, lr=1.5, gamma=0.0, n_pop=1, boundary_mode=mode)
    seeds = np.array([[11], [22], [33], [44]], np.uint64)
    fit = np.array([[1.0], [-1.0], [1.0], [-1.0]], np.float32)
    J = np.arange(n, dtype=np.uint64) + np.uint64(4096)
    step = np.stack([int(fit[k, 0]) * qo.delta(int(seeds[k, 0]), J, 1.5)[0] for k in range(K + 1)])   # [K+1, n]
    outside = (codes[None, :] + step < -8) | (codes[None, :] + step > 7)
    out = qo.update(t, w, None, seeds, fit, K, hp)
    assert np.array_equal(out["gate_replay"], outside[:K].sum(axis=0))
    assert np.array_equal(out["gate_final"], outside[K].astype(np.uint8))
    assert np.array_equal(out["attempted"], (step[K] != 0).astype(np.uint8))
    want_mask = sum(outside[k].astype(np.uint64) << np.uint64(k) for k in range(K + 1))
    assert np.array_equal(out["blocked"], want_mask)
    target = codes + step[K]
    want_w = np.where(outside[K], codes, target) if mode == 0 else np.clip(target, -8, 7)
    assert np.array_equal(out["w_new"], want_w)
    # the case has teeth: blocked steps in the history and in the last generation, and last steps
    # that are non-zero but blocked, zero, and applied
    assert out["gate_replay"].max() >= 2 and out["gate_final"].sum() >= 5
    assert np.any((out["attempted"] == 1) & (out["gate_final"] == 1))
    assert np.any(out["attempted"] == 0) and np.any((out["attempted"] == 1) & (out["gate_final"] == 0))
    # a clamp-shortened step moves the code to the edge and still counts as blocked
    if mode == 1:
        short = outside[K] & (want_w != codes)
        assert short.any() and np.all(out["gate_final"][short] == 1)
    # the history loop alone reports the same history record
    rep = qo.replay_residual(t, w, None, seeds[:K], fit[:K], K, hp)
    assert np.array_equal(rep["gate_replay"], outside[:K].sum(axis=0))
    assert np.array_equal(rep["blocked"], want_mask & np.uint64((1 << K) - 1))


def test_counters_with_the_blocked_signal_carried(qo):
    """gamma = 1 and the same integer set-up: a blocked step stays in the residual, so the next
    generation rounds F delta + e; integer recursion written out here, gate mode."""
    K = 4
    codes = np.tile(np.array([-8, -7, 6, 7], np.int32), 16)
    n = codes.size
    t, w = _tensor(qo, codes, cols=32)
    hp = qo.HParams(sigma=2.0, lr=2.0, gamma=1.0, n_pop=1)
    seeds = np.arange(101, 101 + K + 1, dtype=np.uint64).reshape(K + 1, 1)
    fit = np.ones((K + 1, 1), np.float32)
    J = np.arange(n, dtype=np.uint64)
    e = np.zeros(n, np.int64); replay = np.zeros(n, np.int64); mask = np.zeros(n, np.uint64)
    for k in range(K + 1):
        u = qo.delta(int(seeds[k, 0]), J, 2.0)[0].astype(np.int64) + e        # an integer: its own rounding
        out_of_range = (codes + u < -8) | (codes + u > 7)
        e = np.where(out_of_range, u, 0)
        mask |= out_of_range.astype(np.uint64) << np.uint64(k)
        if k < K:
            replay += out_of_range
    out = qo.update(t, w, None, seeds, fit, K, hp)
    assert np.array_equal(out["gate_replay"], replay) and np.array_equal(out["blocked"], mask)
    assert np.array_equal(out["gate_final"], out_of_range.astype(np.uint8))
    assert np.array_equal(out["attempted"], (u != 0).astype(np.uint8))
    assert np.array_equal(out["e_new"], e.astype(np.float64))
    assert replay.max() >= 3 and np.abs(e).max() >= 4          # carried signal grows past one step


def test_gate_mismatch_count_on_a_true_trajectory_with_a_firing_gate(qo):
    """Sec. 3.3: replay gates against the current weights W_t, the stored-residual run gated against
    W_tau.  INT4 uniform codes, T = 6 steps: the two records of blocked steps differ on a counted set of
    elements; on every other element the replayed residual IS the stored one."""
    n, N, T = 8192, 8, 6
    codes = np.random.default_rng(12).integers(-8, 8, n).astype(np.int32)
    t, _ = _tensor(qo, codes, cols=256, elem_offset=1 << 16)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N)
    seeds, fit = wl.draw_seeds(T, N, stream=41), wl.draw_fitness(T, N, stream=41)
    cur, e_stored, mask_stored, _ = stored_trajectory(qo, t, codes, seeds, fit, hp, 4)
    rep = qo.replay_residual(t, cur, None, seeds, fit, T, hp)
    agree = rep["blocked"] == mask_stored
    mismatches = int((~agree).sum())
    assert np.allclose(rep["e"][agree], e_stored[agree], atol=1e-12)
    # the gate did fire on the trajectory, and replay's view of it is close but not identical
    assert (mask_stored != 0).sum() > 100
    assert 0 < mismatches < 0.15 * n          # uniform codes put 1/8 of the elements on an edge code
    # a mismatch leaves a whole blocked or unblocked step in the residual: it never hides
    assert np.all(np.abs(rep["e"][~agree] - e_stored[~agree]) > 1e-3)
    # with a range the walk cannot reach, nothing is ever blocked and the two runs agree everywhere
    t8, _ = _tensor(qo, codes, bits=8, cols=256, elem_offset=1 << 16)
    cur8, e8, m8, _ = stored_trajectory(qo, t8, codes, seeds, fit, hp, 8)
    rep8 = qo.replay_residual(t8, cur8, None, seeds, fit, T, hp)
    assert not m8.any() and not rep8["blocked"].any() and np.allclose(rep8["e"], e8, atol=1e-12)


def test_weight_unit_sigma_limit_and_extreme_scales(qo):
    """sigma / scale is limited to 2^40 (a zero scale gives +inf -> 2^40, and 2^40 * 0 stays 0): every
    non-zero sample saturates the 4-bit range; the smallest subnormal and the largest finite binary16
    scale follow sigma / scale as they are."""
    rows, cols = 4, 64
    n = rows * cols
    t, w = _tensor(qo, np.zeros(n, np.int32), bits=8, cols=cols, group_size=0)
    J = np.arange(n, dtype=np.uint64)
    hp = qo.HParams(sigma=0.02, lr=1.0, gamma=0.9, n_pop=1, sigma_unit=1)
    scales = np.array([0.0, 2.0 ** -24, 65504.0, 0.01], np.float16)
    assert scales.view(np.uint16).tolist()[:3] == [0x0000, 0x0001, 0x7bff]
    wp = qo.perturb(t, w, scales, 77, hp)
    eps_sign = np.sign(qo.delta(77, J, 1.0, tier=0)[1])                 # sign of eps, from the plain tier
    row0 = wp[:cols]
    assert np.array_equal(row0, np.where(eps_sign[:cols] > 0, 7, -8))    # zero scale: saturated both ways
    assert np.array_equal(row0, qo.delta(77, J[:cols], 2.0 ** 40)[0])
    seff1 = float(np.float32(0.02) / np.float32(2.0 ** -24))
    assert np.array_equal(wp[cols:2 * cols], qo.delta(77, J[cols:2 * cols], seff1)[0])
    seff2 = float(np.float32(0.02) / np.float32(65504.0))
    assert np.array_equal(wp[2 * cols:3 * cols], qo.delta(77, J[2 * cols:3 * cols], seff2)[0])
    assert np.all(wp[2 * cols:3 * cols] == 0)                            # |x| < 2e-6: rounds to 0 here
    # a huge sigma over a small scale overflows the quotient: still 2^40, not inf * 0 = NaN
    hp_big = qo.HParams(sigma=1e29, lr=1.0, gamma=0.9, n_pop=1, sigma_unit=1)
    wp_big = qo.perturb(t, w, np.full(rows, 2.0 ** -24, np.float16), 77, hp_big)
    assert np.array_equal(wp_big, qo.delta(77, J, 2.0 ** 40)[0])
