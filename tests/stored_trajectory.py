"""Algorithm 1 run step by step with the residual kept, written with numpy on top of the oracle's delta (shared by
the CPU pin of the gate-mismatch count and the GPU test of qes_replay_fidelity)."""
import numpy as np


def stored_trajectory(qo, t, codes, seeds, fit, hp, bits):
    """Returns (packed final codes, residual, record of blocked steps (bit s = step s), smallest distance of any
    step's pre-rounding value to a rounding boundary) as they really happen against the evolving weights."""
    n = codes.size
    cur, e, mask = qo.pack(bits, codes), np.zeros(n), np.zeros(n, np.uint64)
    band = np.full(n, 0.5)
    J = np.arange(n, dtype=np.uint64) + np.uint64(t.elem_offset)
    c = float(np.float32(hp.lr)) / (hp.n_pop * float(np.float32(hp.sigma)))
    tc = t.c()
    for s in range(seeds.shape[0]):
        W = qo.unpack(bits, cur, n).astype(np.int64)
        S = sum(float(fit[s, i]) * qo.delta(int(seeds[s, i]), J, hp.sigma)[0] for i in range(hp.n_pop))
        u = c * S + float(np.float32(hp.gamma)) * e
        band = np.minimum(band, np.abs(np.abs(u - np.trunc(u)) - 0.5))
        step = (np.sign(u) * np.floor(np.abs(u) + 0.5)).astype(np.int64)
        if hp.boundary_mode == 0:
            ok = (W + step >= tc.qmin) & (W + step <= tc.qmax)
            applied = np.where(ok, step, 0)
        else:
            applied = np.clip(W + step, tc.qmin, tc.qmax) - W
        mask |= (applied != step).astype(np.uint64) << np.uint64(s)
        e = u - applied
        cur = qo.pack(bits, (W + applied).astype(np.int32))
    return cur, e, mask, band
