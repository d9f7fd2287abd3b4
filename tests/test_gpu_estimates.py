"""The kernels' estimate-then-verify form of the noise sample (special-function estimates first, the exact
fp32 sequence where the estimate cannot settle Eq. 3) must give the contract's delta on every input.
Checked here: the frozen error bound against the device at hand over all 2^24 inputs of each factor;
samples placed on and around rounding decisions; the rate at which the exact sequence is needed."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qes():
    import torch
    from paper_2602_03120_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return binding


def _dev_words(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, np.uint32).view(np.int32)).cuda()


def _guard_width(qes, sigma_eff):
    """E of the verification for a given sigma_eff, as include/qes.h states it."""
    eps, rnd, _ = qes.qes_estimate_bounds()
    need = np.float32(np.float32(sigma_eff * 2.0 ** 24) * np.float32(np.float32(eps) + np.float32(rnd))) + 3.0
    return 1 << min(max(int(np.ceil(np.log2(float(need)))), 4), 24)


def test_estimates_stay_inside_the_frozen_bound_on_every_input(qo, qes):
    """sup over radius words below the limit of R~ * max|trig~ - trig| + |R~ - R| <= eps_bound, measured
    on all 2^24 radius inputs and all 2^24 angle inputs against the oracle's exact factors."""
    import torch
    eps, _, limit = qes.qes_estimate_bounds()
    words = (np.arange(1 << 24, dtype=np.uint64) << 8).astype(np.uint32)
    words |= np.random.default_rng(4).integers(0, 256, size=words.size, dtype=np.uint32)   # low byte: ignored by the
    w = _dev_words(words)                                                                  # contract, seen by the estimate
    R, Cs, Sn = (torch.empty(words.size, dtype=torch.float32, device="cuda") for _ in range(3))
    qes.qes_gaussian_estimates(w, w, R, Cs, Sn)
    Re, Ce, Se = (t.cpu().numpy().astype(np.float64) for t in (R, Cs, Sn))
    Ro, Co, So = (a.astype(np.float64) for a in qo.bm24(words, words))
    trig = max(np.abs(Ce - Co).max(), np.abs(Se - So).max())
    eligible = words < limit
    sup = (Re * trig + np.abs(Re - Ro))[eligible].max()
    print(f"estimates: max trig error {trig:.4g}, sup(R~*dtrig + dR) below the radius limit {sup:.4g} (bound {eps:.4g}), "
          f"radius words excluded {1 - eligible.mean():.3g}")
    assert sup <= eps
    assert np.isfinite(Re).all() and (Re >= 0).all()
    # with the low byte at its extremes too (it moves the estimated angle, never the exact one)
    for low in (0x00, 0xFF):
        wl_ = _dev_words((words & 0xFFFFFF00) | low)
        qes.qes_gaussian_estimates(wl_, wl_, R, Cs, Sn)
        t2 = max(np.abs(Cs.cpu().numpy() - Co).max(), np.abs(Sn.cpu().numpy() - So).max())
        assert (Re * t2 + np.abs(Re - Ro))[eligible].max() <= eps


@pytest.mark.parametrize("sigma_eff", [0.5, 0.25, 2.0, 40.0, 3e-4, 2.0 ** 40])
def test_deltas_on_and_around_rounding_decisions(qo, qes, sigma_eff):
    """For random (radius, angle) words the uniform words are chosen so that the exact rounding sum lands at
    offsets -E-3 .. E+3 (and a few far ones) from a multiple of 2^24 -- where the estimate and the exact value may
    fall on different sides.  Every delta must be the oracle's."""
    import torch
    rng = np.random.default_rng(int(sigma_eff * 1000) % 9973)
    E = _guard_width(qes, sigma_eff)
    n_pairs = 2048 if E <= 4096 else 256
    r0 = rng.integers(0, 1 << 32, n_pairs, dtype=np.uint64).astype(np.uint32)
    r1 = rng.integers(0, 1 << 32, n_pairs, dtype=np.uint64).astype(np.uint32)
    r0[:8] = [0, 0xFF, 0x100, 0xFFFF7FFF, 0xFFFF8000, 0xFFFFFF00, 0xFFFFFFFF, 0x80000000]   # radius extremes, limit edges
    r1[:8] = [0, 0x40000000, 0x80000000, 0xC0000000, 0x3FFFFFFF, 0x7FFFFFFF, 0xFFFFFFFF, 0x00000100]
    R, c, s = qo.bm24(r0, r1)
    rho = np.float32(sigma_eff) * R                                          # fp32 products, as the contract states
    if E <= 4096:
        offs = np.concatenate([np.arange(-E - 3, E + 4), [-(1 << 23), 1 << 22, 12345]])
    else:
        offs = np.concatenate([np.arange(-40, 41), rng.integers(-(1 << 23), 1 << 23, 80),
                               [E - 1, E, E + 1, -E - 1, -E, -E + 1, 2 * E, -2 * E]])
    offs = offs.astype(np.int64)
    cols = []
    for trig in (c, s):
        y = -(rho * trig).astype(np.float64) * 2.0 ** 24                     # exact: a power-of-two multiple of an fp32
        fl = np.floor(np.clip(y, -9.0 * 2 ** 24, 9.0 * 2 ** 24)).astype(np.int64)
        v = (offs[None, :] - fl[:, None]) % (1 << 24)                        # floor(y) + v = offs (mod 2^24)
        cols.append(((v << 8) | rng.integers(0, 256, v.shape)).astype(np.uint32))
    m = offs.size
    R0, R1 = np.repeat(r0, m), np.repeat(r1, m)
    R2, R3 = cols[0].reshape(-1), cols[1].reshape(-1)
    de = torch.empty(R0.size, dtype=torch.int8, device="cuda"); do = torch.empty_like(de)
    ver = torch.empty(R0.size, dtype=torch.uint8, device="cuda")
    qes.qes_pair_deltas(_dev_words(R0), _dev_words(R1), _dev_words(R2), _dev_words(R3), sigma_eff, de, do, ver)
    want_e, want_o = qo.pair_deltas(R0, R1, R2, R3, sigma_eff)
    got_e, got_o, ver = de.cpu().numpy(), do.cpu().numpy(), ver.cpu().numpy()
    assert np.array_equal(got_e, want_e), f"{(got_e != want_e).sum()} even deltas differ"
    assert np.array_equal(got_o, want_o), f"{(got_o != want_o).sum()} odd deltas differ"
    # the planted offsets do straddle decisions, and samples right on one went through the exact sequence
    if sigma_eff <= 0.5:                                                     # no sample saturates the 4-bit range here
        flips = (np.diff(want_e.reshape(n_pairs, m)[:, :2 * E + 7], axis=1) != 0).sum(axis=1)
        assert (flips >= 1).mean() > 0.99                                    # delta steps between offsets -1 and 0
    on_decision = np.repeat(np.abs(offs)[None, :] <= 1, n_pairs, axis=0).reshape(-1)
    assert ver[on_decision].all()
    if E <= 256:
        far = np.repeat((np.abs(offs) > 4 * E)[None, :], n_pairs, axis=0).reshape(-1) & (R0 < qes.qes_estimate_bounds()[2])
        assert ver[far].mean() < 0.05                                       # far from a decision the estimate settles it
    assert ver[np.repeat(r0 >= qes.qes_estimate_bounds()[2], m)].all()       # radius words past the limit: always exact


def test_exact_sequence_rate_and_full_agreement_on_random_words(qo, qes):
    """2^22 random word quadruples at sigma = 0.5 (the benchmark's value): every delta is the oracle's, and the
    exact sequence is needed for a few pairs in 10^5."""
    import torch
    n = 1 << 22
    rng = np.random.default_rng(2024)
    r = [rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32) for _ in range(4)]
    de = torch.empty(n, dtype=torch.int8, device="cuda"); do = torch.empty_like(de)
    ver = torch.empty(n, dtype=torch.uint8, device="cuda")
    qes.qes_pair_deltas(*(_dev_words(x) for x in r), 0.5, de, do, ver)
    want_e, want_o = qo.pair_deltas(*r, 0.5)
    assert np.array_equal(de.cpu().numpy(), want_e) and np.array_equal(do.cpu().numpy(), want_o)
    rate = float(ver.cpu().numpy().mean())
    E = _guard_width(qes, 0.5)
    expected = 2 * (2 * E) / 2.0 ** 24 + (2.0 ** 32 - qes.qes_estimate_bounds()[2]) / 2.0 ** 32
    print(f"exact sequence needed for {rate:.3g} of the pairs at sigma = 0.5 (E = {E}; expected {expected:.3g})")
    assert E == 128 and 0.3 * expected < rate < 3 * expected
