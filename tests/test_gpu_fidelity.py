"""qes_replay_fidelity against the oracle: the gate-mismatch count of Stateless Seed Replay on a true
stored-residual trajectory (Sec. 3.3), where the gate fires and where it cannot."""
import numpy as np
import pytest

from paper_2602_03120_b200 import workloads as wl
from stored_trajectory import stored_trajectory

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qes():
    import torch
    from paper_2602_03120_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return binding


def _dev(a):
    import torch
    a = np.ascontiguousarray(a)
    return torch.from_numpy(a.view(np.int64) if a.dtype == np.uint64 else a).cuda()


@pytest.mark.parametrize("bits,rows,cols,N,T,mode,sigma,lo,hi", [
    (4, 61, 416, 8, 6, 0, 0.5, -8, 8), (4, 33, 256, 6, 9, 1, 0.5, -8, 8), (8, 40, 256, 8, 8, 0, 0.5, -64, 64),
    (4, 17, 512, 4, 33, 0, 1.5, -8, 8), (8, 9, 128, 5, 3, 0, 0.5, -128, 128)])
def test_gate_mismatch_count_matches_the_oracle(qo, qes, bits, rows, cols, N, T, mode, sigma, lo, hi):
    """Codes uniform in [lo, hi): the INT4 cases put an eighth of the elements on an edge code, so records of blocked
    steps do differ between the true trajectory and its replay; the INT8 case in [-64, 64) can never reach an edge."""
    import torch
    n = rows * cols
    codes = np.random.default_rng([bits, rows, T]).integers(lo, hi, n).astype(np.int32)
    off = 32 * 4000
    to = qo.Tensor(bits=bits, rows=rows, cols=cols, elem_offset=off)
    tg = qes.TensorDesc(bits=bits, rows=rows, cols=cols, elem_offset=off)
    kw = dict(sigma=sigma, lr=1.0, gamma=0.9, n_pop=N, boundary_mode=mode)
    ho, hg = qo.HParams(**kw), qes.HParams(**kw)
    seeds, fit = wl.draw_seeds(T, N, stream=70 + T), wl.draw_fitness(T, N, stream=70 + T)
    # oracle: the stored-residual run, then the history loop against its final weights
    cur, e_true, mask_true, band_true = stored_trajectory(qo, to, codes, seeds, fit, ho, bits)
    rep = qo.replay_residual(to, cur, None, seeds, fit, T, ho)
    differ = rep["blocked"] != mask_true
    near = (band_true < 1e-5) | (rep["band"] < 1e-5)          # fp32 may round these the other way
    # library
    packed = qo.pack(bits, codes)
    w0, w_end = _dev(packed), _dev(np.zeros_like(packed))
    counts = torch.zeros(4, dtype=torch.int64, device="cuda")
    qes.qes_replay_fidelity(tg, w0, w_end, None, _dev(seeds), _dev(fit), T, hg, counts)
    got = counts.cpu().numpy()
    slack = int(near.sum())
    assert abs(int(got[0]) - int(differ.sum())) <= slack, (got, int(differ.sum()), slack)
    assert abs(int(got[1]) - int((mask_true != 0).sum())) <= slack
    assert abs(int(got[2]) - int((np.abs(rep["e"] - e_true) > 1e-5).sum())) <= slack
    if mode == 0:
        assert got[2] <= got[0]       # gate: equal records give equal residuals (a clamp may shorten by different amounts)
    end = qo.unpack(bits, w_end.cpu().numpy(), n)
    want_end = qo.unpack(bits, cur, n)
    assert not np.any((end != want_end) & ~near)
    assert abs(int(got[3]) - int((want_end != codes).sum())) <= slack
    assert np.array_equal(w0.cpu().numpy(), packed)
    if hi - lo == 16:
        assert got[0] > 0 and got[1] > got[0] / 4                 # the gate fires, replay sees it slightly differently
    if bits == 8 and hi == 64:
        assert got[0] == 0 and got[1] == 0 and got[2] == 0 and got[3] > 0
    # counts are added to, and the final weights may replace the start in place
    qes.qes_replay_fidelity(tg, w0, w0, None, _dev(seeds), _dev(fit), T, hg, counts)
    assert np.array_equal(counts.cpu().numpy(), 2 * got) and torch.equal(w0, w_end)


def test_final_weights_are_the_stored_residual_chain_of_qes_update(qo, qes):
    """Pass (1) of the fidelity call is Algorithm 1 as qes_update runs it with a stored residual, step by step."""
    import torch
    rows, cols, N, T = 48, 512, 8, 5
    packed = np.random.default_rng(3).integers(0, 256, rows * cols // 2, dtype=np.uint8)
    tg = qes.TensorDesc(bits=4, rows=rows, cols=cols, elem_offset=64)
    hg = qes.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N)
    seeds, fit = wl.draw_seeds(T, N, stream=81), wl.draw_fitness(T, N, stream=81)
    w, e = _dev(packed), torch.zeros(rows * cols, dtype=torch.float32, device="cuda")
    for s in range(T):
        qes.qes_update(tg, w, None, _dev(seeds[s:s + 1]), _dev(fit[s:s + 1]), 0, e, hg)
    w_end = _dev(np.zeros_like(packed))
    counts = torch.zeros(4, dtype=torch.int64, device="cuda")
    qes.qes_replay_fidelity(tg, _dev(packed), w_end, None, _dev(seeds), _dev(fit), T, hg, counts)
    assert torch.equal(w_end, w)
    # and pass (2) is qes_replay_residual on those final weights: residuals differ exactly where counted
    e_rep = torch.empty_like(e)
    qes.qes_replay_residual(tg, w, None, _dev(seeds), _dev(fit), T, hg, e_rep)
    assert int(((e_rep - e).abs() > 1e-5).sum()) == int(counts[2])
