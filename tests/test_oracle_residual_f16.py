"""Pins for Algorithm 1 with the residual stored in binary16 ("Initialize: Residuals e_0 <- 0 (FP16)")."""
import numpy as np

from paper_2602_03120_b200 import workloads as wl


def _setup(qo, n=4096, seed=3):
    codes = np.random.default_rng(seed).integers(-40, 40, n)
    t = qo.Tensor(bits=8, rows=n // 64, cols=64)
    return t, qo.pack(8, codes.astype(np.int32)), codes


def test_representable_residuals_give_the_fp32_result(qo):
    t, w, _ = _setup(qo)
    e16 = np.random.default_rng(1).uniform(-0.5, 0.5, 4096).astype(np.float16)
    seeds, fit = wl.draw_seeds(1, 8, stream=61), wl.draw_fitness(1, 8, stream=61)
    kw = dict(sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    a = qo.update(t, w, None, seeds, fit, 0, qo.HParams(**kw, residual_f16=1), residual_in=e16)
    b = qo.update(t, w, None, seeds, fit, 0, qo.HParams(**kw), residual_in=e16.astype(np.float32))
    assert np.array_equal(a["w_new"], b["w_new"]) and np.array_equal(a["e_new"], b["e_new"])
    assert np.any(a["w_new"] != qo.unpack(8, w, 4096))


def test_fp16_storage_tracks_fp32_storage_within_its_rounding(qo):
    """T steps of Algorithm 1, residual rounded to binary16 after every step, against fp32 storage: each
    store moves e by at most half a binary16 spacing (2^-12 for |e| <= 1/2), decayed by gamma afterwards, so
    the two residuals stay within 2^-12 / (1 - gamma) and the codes agree wherever no pre-rounding value
    came that close to a rounding boundary."""
    t, w0, codes = _setup(qo, seed=4)
    T, N, gamma = 12, 8, 0.9
    kw = dict(sigma=0.5, lr=0.6, gamma=gamma, n_pop=N)
    w32, w16 = w0.copy(), w0.copy()
    e32 = np.zeros(4096, np.float32)
    e16 = np.zeros(4096, np.uint16)
    bound = 2.0 ** -12 / (1.0 - gamma)
    clean = np.ones(4096, bool)
    for step in range(T):
        seeds, fit = wl.draw_seeds(1, N, stream=70 + step), wl.draw_fitness(1, N, stream=70 + step)
        a = qo.update(t, w32, None, seeds, fit, 0, qo.HParams(**kw), residual_in=e32)
        b = qo.update(t, w16, None, seeds, fit, 0, qo.HParams(**kw, residual_f16=1), residual_in=e16)
        clean &= (a["band"] > bound + 1e-6) & (a["gate_final"] == 0) & (b["gate_final"] == 0)
        w32, e32 = qo.pack(8, a["w_new"]), a["e_new"].astype(np.float32)
        w16, e16 = qo.pack(8, b["w_new"]), qo.to_half(b["e_new"])
        stored = e16.view(np.float16).astype(np.float64)
        assert np.abs(stored - b["e_new"]).max() <= 2.0 ** -12 + 1e-12          # one store: half a spacing
        assert np.abs(stored[clean] - e32[clean]).max() <= bound
        assert np.abs(stored[clean]).max() <= 0.5 + 2.0 ** -12
    assert clean.mean() > 0.5
    assert np.array_equal(qo.unpack(8, w16, 4096)[clean], qo.unpack(8, w32, 4096)[clean])
    assert np.any(qo.unpack(8, w32, 4096) != codes)
