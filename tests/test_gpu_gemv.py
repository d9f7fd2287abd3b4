"""The batch-1 weight read (qes_gemv) and the same read with the member's perturbation generated inside it
(qes_gemv_perturbed) against float64 sums over the oracle's codes; the in-read perturbation must give exactly
the codes qes_perturb stores (Algorithm 1, member loop; Eqs. 3-4)."""
import numpy as np
import pytest

from paper_2602_03120_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qes():
    import torch
    from paper_2602_03120_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return binding


def _reference(codes, scales, x, rows, cols):
    """float64 row sums, and the 2-norm of each row's terms (the scale of the fp16 accumulation error)."""
    q = codes.reshape(rows, cols).astype(np.float64)
    s = scales.astype(np.float64).reshape(rows, -1)
    s_full = np.repeat(s, cols // s.shape[1], axis=1)
    terms = q * s_full * x.astype(np.float64)[None, :]
    return terms.sum(axis=1), np.sqrt((terms ** 2).sum(axis=1))


@pytest.mark.parametrize("rows,cols,group,off,sigma,mode,unit", [
    (37, 352, 32, 0, 0.5, 0, 0), (5, 3584, 128, 32 * 1000, 0.5, 1, 0), (19, 1024, 0, (1 << 34) - 4096, 2.0, 0, 0),
    (9, 256, 64, 64, 0.012, 0, 1), (1, 32, 32, 0, 0.5, 0, 0)])
def test_gemv_plain_and_perturbed_small_shapes(qo, qes, rows, cols, group, off, sigma, mode, unit):
    import torch
    rng = np.random.default_rng([rows, cols])
    n = rows * cols
    packed = rng.integers(0, 256, n // 2, dtype=np.uint8)
    scales = rng.lognormal(-4.0, 0.3, size=rows * (cols // group) if group else rows).astype(np.float16)
    x = rng.standard_normal(cols).astype(np.float16)
    to = qo.Tensor(bits=4, rows=rows, cols=cols, group_size=group, elem_offset=off)
    tg = qes.TensorDesc(bits=4, rows=rows, cols=cols, group_size=group, elem_offset=off)
    kw = dict(sigma=sigma, lr=1.0, gamma=0.9, n_pop=4, boundary_mode=mode, sigma_unit=unit)
    ho, hg = qo.HParams(**kw), qes.HParams(**kw)
    w, sc, xd = (torch.from_numpy(a).cuda() for a in (packed, scales, x))
    y = torch.full((rows,), 7.0, dtype=torch.float32, device="cuda")
    qes.qes_gemv(tg, w, sc, xd, y)
    want, norm = _reference(qo.unpack(4, packed, n), scales, x, rows, cols)
    assert np.all(np.abs(y.cpu().numpy() - want) <= 5e-3 * norm + 1e-7)
    seed = 0xABCD_0000_1234 + rows
    yp = torch.empty_like(y)
    qes.qes_gemv_perturbed(tg, w, sc, seed, hg, xd, yp)
    pert = qo.perturb(to, packed, scales if unit else None, seed, ho)
    want_p, norm_p = _reference(pert, scales, x, rows, cols)
    assert np.all(np.abs(yp.cpu().numpy() - want_p) <= 5e-3 * norm_p + 1e-7)
    assert np.any(pert != qo.unpack(4, packed, n))
    # the same codes as the stored perturbed copy: identical arithmetic on identical codes
    wp = torch.empty_like(w)
    qes.qes_perturb(tg, w, wp, sc if unit else None, seed, hg)
    y2 = torch.empty_like(y)
    qes.qes_gemv(tg, wp, sc, xd, y2)
    assert torch.equal(y2, yp)
    assert torch.equal(w.cpu(), torch.from_numpy(packed))          # the read leaves the weights alone


def test_gemv_on_a_7b_k_proj(qo, qes):
    """One k_proj of the 7B-shaped set (512 x 3584, group 128) at its place in the model: plain and perturbed reads
    against float64 sums over the oracle's (perturbed) codes."""
    import torch
    cfg = wl.WORKLOADS["decoder7b_int4"]
    ti = 8                                                     # layers.1.k_proj
    t = cfg.tensors[ti]
    assert (t.rows, t.cols) == (512, 3584)
    packed, scales = wl.draw_codes(cfg, ti), wl.draw_scales(cfg, ti)
    x = np.random.default_rng(17).standard_normal(t.cols).astype(np.float16)
    to = qo.Tensor(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
    tg = qes.TensorDesc(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
    kw = dict(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    ho, hg = qo.HParams(**kw), qes.HParams(**kw)
    w, sc, xd = (torch.from_numpy(a).cuda() for a in (packed, scales, x))
    y, yp = (torch.empty(t.rows, dtype=torch.float32, device="cuda") for _ in range(2))
    seed = int(wl.draw_seeds(1, 1, stream=55)[0, 0])
    qes.qes_gemv(tg, w, sc, xd, y)
    qes.qes_gemv_perturbed(tg, w, sc, seed, hg, xd, yp)
    want, norm = _reference(qo.unpack(4, packed, t.numel), scales, x, t.rows, t.cols)
    pert = qo.perturb(to, packed, None, seed, ho)
    want_p, norm_p = _reference(pert, scales, x, t.rows, t.cols)
    err, err_p = np.abs(y.cpu().numpy() - want) / norm, np.abs(yp.cpu().numpy() - want_p) / norm_p
    print(f"k_proj read: max |y - y64| / ||terms|| plain {err.max():.2e}, perturbed {err_p.max():.2e}; "
          f"{(pert != qo.unpack(4, packed, t.numel)).mean():.3f} of the codes perturbed")
    assert err.max() <= 5e-3 and err_p.max() <= 5e-3
    assert np.abs(want - want_p).max() > 20 * np.abs(yp.cpu().numpy() - want_p).max()   # the perturbation is what the read sees
