"""The seed/reward window of Algorithm 2 (host bookkeeping) and the checkpoint/resume property it gives:
the whole optimizer state is the packed weights plus a few kilobytes of history."""
import numpy as np
import pytest

from paper_2602_03120_b200 import workloads as wl
from paper_2602_03120_b200.history import SeedHistory


def test_window_order_size_and_serialisation():
    K, N = 3, 4
    h = SeedHistory(K, N)
    gens = [(wl.draw_seeds(1, N, stream=s)[0], wl.draw_fitness(1, N, stream=s)[0]) for s in range(6)]
    for t, (s, f) in enumerate(gens):
        seeds, fit, k = h.tables(s, f)
        assert k == min(t, K) and seeds.size == (k + 1) * N and fit.size == (k + 1) * N
        want = gens[max(0, t - K):t + 1]                       # oldest first, the current generation last
        assert np.array_equal(seeds, np.concatenate([g[0] for g in want]))
        assert np.array_equal(fit, np.concatenate([g[1] for g in want]))
        h2 = SeedHistory.from_bytes(h.to_bytes())
        assert all(np.array_equal(a, b) for a, b in zip(h2.tables(s, f)[:2], (seeds, fit)))
        h.push(s, f)
    assert len(h) == K and h.nbytes == K * N * 12
    big = SeedHistory(50, 50)
    for _ in range(60):
        big.push(np.zeros(50, np.uint64), np.zeros(50, np.float32))
    assert big.nbytes == 30_000                                # the paper's "≈29.7 KB" optimizer state
    with pytest.raises(ValueError):
        h.push(np.zeros(3, np.uint64), np.zeros(N, np.float32))
    pairs = SeedHistory(2, 8, seeds_per_generation=4)          # antithetic pairs: one seed per pair
    pairs.push(np.arange(4, dtype=np.uint64), np.zeros(8, np.float32))
    assert pairs.tables(np.arange(4, dtype=np.uint64), np.ones(8, np.float32))[0].size == 8


def test_resume_from_history_and_weights_is_bit_identical(qo):
    """T steps of the stateless update in one go equal T/2 steps, a round trip of (weights, history) through
    bytes, and T/2 more steps (oracle; the GPU suite repeats this through the library)."""
    N, K, T = 4, 3, 6
    t = qo.Tensor(bits=4, rows=8, cols=64)
    w0 = np.random.default_rng(2).integers(0, 256, 256, dtype=np.uint8)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N)
    gens = [(wl.draw_seeds(1, N, stream=500 + s)[0], wl.draw_fitness(1, N, stream=500 + s)[0]) for s in range(T)]

    def run(w, hist, steps):
        for s, f in steps:
            seeds, fit, k = hist.tables(s, f)
            w = qo.pack(4, qo.update(t, w, None, seeds, fit, k, hp)["w_new"])
            hist.push(s, f)
        return w, hist

    w_full, _ = run(w0, SeedHistory(K, N), gens)
    w_half, hist = run(w0, SeedHistory(K, N), gens[:T // 2])
    blob_w, blob_h = w_half.tobytes(), hist.to_bytes()
    w_res, _ = run(np.frombuffer(blob_w, np.uint8).copy(), SeedHistory.from_bytes(blob_h), gens[T // 2:])
    assert np.array_equal(w_full, w_res) and not np.array_equal(w_full, w0)
