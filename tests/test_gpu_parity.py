"""Parity of the CUDA library (through its C ABI) against the CPU oracle, element by element.

Rules: packed codes bit-exact, except elements whose pre-rounding value u lies within
1e-5 of a rounding boundary in any generation (counted, reported, never silently skipped);
residuals within 1e-5 absolute on the remaining elements.  qes_perturb has no such band: exact.
"""
import numpy as np
import pytest

from paper_2602_03120_b200 import workloads as wl

pytestmark = pytest.mark.gpu

BAND = 1e-5
TOL = 1e-5


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
    if a.dtype == np.uint64:
        a = a.view(np.int64)
    return torch.from_numpy(a).cuda()


def _host(t):
    return t.cpu().numpy()


def _case(qo, qes, bits, rows, cols, group=0, off=0, qmin=None, qmax=None, seed=0):
    n = rows * cols
    rng = np.random.default_rng([seed, rows, cols])
    packed = rng.integers(0, 256, size=n if bits == 8 else n // 2, dtype=np.uint8)
    if qmin is not None:   # keep codes inside a narrower range
        codes = np.clip(qo.unpack(bits, packed, n), qmin, qmax)
        packed = qo.pack(bits, codes)
    to = qo.Tensor(bits=bits, rows=rows, cols=cols, group_size=group, elem_offset=off, qmin=qmin, qmax=qmax)
    tg = qes.TensorDesc(bits=bits, rows=rows, cols=cols, group_size=group, elem_offset=off, qmin=qmin, qmax=qmax)
    n_scales = rows * (cols // group) if group else rows
    scales = rng.lognormal(-4.0, 0.3, size=n_scales).astype(np.float16)
    return to, tg, packed, scales


def _codes_at(qo, bits, packed, idx):
    """Codes of the sampled elements; idx is made of whole, aligned 32-element words (wl.sample_elements)."""
    per_word = 32 if bits == 8 else 16
    words = idx.reshape(-1, 32)[:, 0] // 32
    compact = np.ascontiguousarray(packed.reshape(-1, per_word)[words]).reshape(-1)
    return qo.unpack(bits, compact, idx.size)


def _hp(qo, qes, **kw):
    return qo.HParams(**kw), qes.HParams(**kw)


def _compare_update(qo, packed_gpu, bits, ref, what=""):
    got = qo.unpack(bits, packed_gpu, ref["w_new"].size)
    near = ref["band"] < BAND
    bad = (got != ref["w_new"]) & ~near
    assert not bad.any(), f"{what}: {bad.sum()} codes differ outside the rounding band (near-band: {near.sum()})"
    # inside the band either rounding is acceptable, but it must be one of the two neighbours
    assert np.all(np.abs(got[near] - ref["w_new"][near]) <= 1)
    return int(near.sum())


@pytest.mark.parametrize("bits,rows,cols,off", [(4, 37, 352, 0), (8, 21, 160, 96), (4, 1, 32, 0),
                                                (4, 9, 4096, (1 << 34) + 64), (8, 3, 64, (1 << 40))])
def test_perturb_bit_exact(qo, qes, bits, rows, cols, off):
    to, tg, packed, _ = _case(qo, qes, bits, rows, cols, off=off)
    for mode in (0, 1):
        for sigma in (0.5, 2.0):          # 2.0 compiles in the 4-bit limit on delta
            ho, hg = _hp(qo, qes, sigma=sigma, lr=1.0, gamma=0.9, n_pop=1, boundary_mode=mode)
            seed = 0xC0FFEE_0000_0000 + rows
            w_in = _dev(packed); w_out = _dev(np.zeros_like(packed))
            qes.qes_perturb(tg, w_in, w_out, None, seed, hg)
            ref = qo.perturb(to, packed, None, seed, ho)
            assert np.array_equal(_host(w_out), qo.pack(bits, ref))
            assert np.array_equal(_host(w_in), packed)
            qes.qes_perturb(tg, w_in, w_in, None, seed, hg)     # exact aliasing is allowed
            assert np.array_equal(_host(w_in), qo.pack(bits, ref))
    assert np.any(ref != qo.unpack(bits, packed, rows * cols))


@pytest.mark.parametrize("bits,rows,cols,group,N,K,mode", [
    (4, 67, 1024, 128, 8, 4, 0), (4, 5, 96, 32, 3, 0, 0), (8, 33, 544, 0, 5, 3, 0),
    (4, 19, 640, 64, 7, 6, 1), (8, 1, 32, 0, 1, 1, 1)])
def test_stateless_update_and_replay(qo, qes, bits, rows, cols, group, N, K, mode):
    import torch
    to, tg, packed, scales = _case(qo, qes, bits, rows, cols, group=group, off=32 * 1001)
    ho, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=N, boundary_mode=mode)
    seeds, fit = wl.draw_seeds(K + 1, N, stream=rows), wl.draw_fitness(K + 1, N, stream=rows)
    w = _dev(packed); stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), K, None, hg, stats=stats)
    ref = qo.update(to, packed, None, seeds, fit, K, ho)
    n_near = _compare_update(qo, _host(w), bits, ref, "stateless update")
    st = _host(stats)
    far = ref["band"] >= BAND
    changed = (ref["w_new"] != qo.unpack(bits, packed, rows * cols))
    assert abs(int(st[0]) - int(changed.sum())) <= n_near
    assert abs(int(st[1]) - int(ref["gate_final"].sum())) <= n_near
    assert abs(int(st[2]) - int(ref["gate_replay"].sum())) <= n_near * max(K, 1)
    assert abs(int(st[3]) - int(ref["attempted"].sum())) <= n_near
    # history loop alone
    res = torch.full((rows * cols,), 7.0, dtype=torch.float32, device="cuda")
    qes.qes_replay_residual(tg, _dev(packed), None, _dev(seeds[:K]), _dev(fit[:K]), K, hg, res)
    rr = qo.replay_residual(to, packed, None, seeds[:K], fit[:K], K, ho)
    farr = rr["band"] >= BAND
    assert np.abs(_host(res).astype(np.float64) - rr["e"])[farr].max(initial=0.0) <= TOL
    assert farr.mean() > 0.99


def test_stored_residual_step(qo, qes):
    import torch
    to, tg, packed, _ = _case(qo, qes, 4, 41, 288)
    ho, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    n = 41 * 288
    e_in = np.random.default_rng(0).uniform(-0.5, 0.5, n).astype(np.float32)
    seeds, fit = wl.draw_seeds(1, 8, stream=77), wl.draw_fitness(1, 8, stream=77)
    w = _dev(packed); e = _dev(e_in)
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), 0, e, hg)
    ref = qo.update(to, packed, None, seeds, fit, 0, ho, residual_in=e_in)
    _compare_update(qo, _host(w), 4, ref, "stored residual")
    far = ref["band"] >= BAND
    assert np.abs(_host(e).astype(np.float64) - ref["e_new"])[far].max() <= TOL


def test_weight_unit_sigma_reads_group_scales(qo, qes):
    for bits, rows, cols, group in ((4, 23, 512, 128), (4, 7, 256, 64), (8, 29, 96, 0)):
        to, tg, packed, scales = _case(qo, qes, bits, rows, cols, group=group)
        kw = dict(sigma=0.012, lr=1.0, gamma=0.9, n_pop=6, sigma_unit=1)
        ho, hg = _hp(qo, qes, **kw)
        seeds, fit = wl.draw_seeds(3, 6, stream=5), wl.draw_fitness(3, 6, stream=5)
        w = _dev(packed)
        qes.qes_update(tg, w, _dev(scales), _dev(seeds), _dev(fit), 2, None, hg)
        ref = qo.update(to, packed, scales, seeds, fit, 2, ho)
        _compare_update(qo, _host(w), bits, ref, "weight-unit sigma")
        wp = _dev(np.zeros_like(packed))
        qes.qes_perturb(tg, _dev(packed), wp, _dev(scales), 99, hg)
        assert np.array_equal(_host(wp), qo.pack(bits, qo.perturb(to, packed, scales, 99, ho)))


def test_symmetric_grid_range(qo, qes):
    """App. A grid: codes in [-(2^(B-1)-1), 2^(B-1)-1]."""
    to, tg, packed, _ = _case(qo, qes, 4, 16, 256, qmin=-7, qmax=7)
    ho, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    seeds, fit = wl.draw_seeds(3, 8, stream=6), wl.draw_fitness(3, 8, stream=6)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), 2, None, hg)
    ref = qo.update(to, packed, None, seeds, fit, 2, ho)
    _compare_update(qo, _host(w), 4, ref, "symmetric grid")
    got = qo.unpack(4, _host(w), 16 * 256)
    assert got.min() >= -7 and got.max() <= 7


def test_split_invariance_and_determinism(qo, qes):
    to, tg, packed, _ = _case(qo, qes, 4, 64, 256, off=1 << 21)
    _, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    seeds, fit = _dev(wl.draw_seeds(4, 8)), _dev(wl.draw_fitness(4, 8))
    whole = _dev(packed)
    qes.qes_update(tg, whole, None, seeds, fit, 3, None, hg)
    again = _dev(packed)
    qes.qes_update(tg, again, None, seeds, fit, 3, None, hg)
    assert np.array_equal(_host(whole), _host(again))
    half = 32 * 256
    top = qes.TensorDesc(bits=4, rows=32, cols=256, elem_offset=1 << 21)
    bot = qes.TensorDesc(bits=4, rows=32, cols=256, elem_offset=(1 << 21) + half)
    a, b = _dev(packed[:half // 2]), _dev(packed[half // 2:])
    qes.qes_update(top, a, None, seeds, fit, 3, None, hg)
    qes.qes_update(bot, b, None, seeds, fit, 3, None, hg)
    assert np.array_equal(np.concatenate([_host(a), _host(b)]), _host(whole))


def test_empty_history_and_zero_fitness(qo, qes):
    import torch
    to, tg, packed, _ = _case(qo, qes, 4, 4, 128)
    _, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=4)
    res = torch.full((512,), 3.0, dtype=torch.float32, device="cuda")
    qes.qes_replay_residual(tg, _dev(packed), None, None, None, 0, hg, res)
    assert np.all(_host(res) == 0.0)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(wl.draw_seeds(3, 4)), _dev(np.zeros((3, 4), np.float32)), 2, None, hg)
    assert np.array_equal(_host(w), packed)


def test_config1_full_matrix(qo, qes):
    """Benchmark configuration 1 in full: 4096x4096 INT4, N = 8, K = 4, every element compared."""
    cfg = wl.WORKLOADS["matrix4096_int4"]
    t = cfg.tensors[0]
    packed = wl.draw_codes(cfg, 0)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)
    kw = dict(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    ho, hg = _hp(qo, qes, **kw)
    to = qo.Tensor(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size)
    tg = qes.TensorDesc(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), cfg.K, None, hg)
    ref = qo.update(to, packed, None, seeds, fit, cfg.K, ho)
    n_near = _compare_update(qo, _host(w), 4, ref, "config 1")
    print(f"config 1: {t.numel} elements, {n_near} inside the 1e-5 rounding band")
    assert n_near < 1e-3 * t.numel
    assert (ref["w_new"] != qo.unpack(4, packed, t.numel)).mean() > 0.01


@pytest.mark.parametrize("name", ["decoder1p5b_int4", "decoder7b_int4", "decoder7b_int8", "decoder8b_int4"])
def test_full_size_tensors_sampled(qo, qes, name):
    """Full-size tensors of the large configurations in the benchmark's launch configuration (one call per
    tensor, the configuration's N and K), oracle on sampled 32-element words incl. first and last."""
    cfg = wl.WORKLOADS[name]
    kw = dict(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    ho, hg = _hp(qo, qes, **kw)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)
    ds, df = _dev(seeds), _dev(fit)
    per_tensor = 2048 if cfg.K <= 16 else 256
    picks = [1, 6, len(cfg.tensors) - 1] if cfg.K <= 16 else [len(cfg.tensors) - 6]   # k_proj, down_proj, last / one k_proj
    total_near = 0
    for ti in picks:
        t = cfg.tensors[ti]
        packed = wl.draw_codes(cfg, ti)
        to = qo.Tensor(bits=cfg.bits, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
        tg = qes.TensorDesc(bits=cfg.bits, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
        w = _dev(packed)
        qes.qes_update(tg, w, None, ds, df, cfg.K, None, hg)
        idx = wl.sample_elements(t.numel, per_tensor, stream=ti)
        ref = qo.update(to, packed, None, seeds, fit, cfg.K, ho, idx=idx)
        got = _codes_at(qo, cfg.bits, _host(w), idx)
        near = ref["band"] < BAND
        assert not np.any((got != ref["w_new"]) & ~near), f"{name} tensor {ti}"
        total_near += int(near.sum())
        # properties that hold at any size: range, and untouched where the oracle sample is untouched
        assert got.min() >= cfg.qmin and got.max() <= cfg.qmax
        # Algorithm 1's member loop on the same full-size tensor: bit-exact on the sample
        wp = _dev(np.zeros_like(packed))
        qes.qes_perturb(tg, _dev(packed), wp, None, int(seeds[-1, ti % cfg.n_pop]), hg)
        want = qo.perturb(to, packed, None, int(seeds[-1, ti % cfg.n_pop]), ho, idx=idx)
        assert np.array_equal(_codes_at(qo, cfg.bits, _host(wp), idx), want), f"{name} tensor {ti}: perturb"
    print(f"{name}: near-band sampled elements {total_near}")


def test_perturb_delta_is_the_delta_the_update_sums(qo, qes):
    to, tg, packed, _ = _case(qo, qes, 8, 8, 128)
    packed = np.zeros_like(packed)           # far from the boundary: perturb output is delta itself
    ho, hg = _hp(qo, qes, sigma=1.0, lr=1.0, gamma=0.0, n_pop=1)
    seed = 424242
    wp = _dev(np.zeros_like(packed))
    qes.qes_perturb(tg, _dev(packed), wp, None, seed, hg)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(np.array([[seed]], np.uint64)), _dev(np.array([[1.0]], np.float32)), 0, None, hg)
    assert np.array_equal(_host(wp), _host(w))
    assert np.array_equal(qo.unpack(8, _host(wp), 1024), qo.delta(seed, np.arange(1024, dtype=np.uint64), 1.0)[0])


def test_gaussian_factors_bit_identical_on_the_whole_domain(qo, qes):
    """Every one of the 2^24 radii and 2^24 (cos, sin) pairs of the noise contract: the kernel's fp32
    sequence (its own square root, its own argument reduction) against the oracle's, bit for bit."""
    import torch
    words = (np.arange(1 << 24, dtype=np.uint64) << 8).astype(np.uint32)
    words |= np.random.default_rng(3).integers(0, 256, size=words.size, dtype=np.uint32)   # low byte is unused
    w = torch.from_numpy(words.view(np.int32)).cuda()
    R, Cs, Sn = (torch.empty(words.size, dtype=torch.float32, device="cuda") for _ in range(3))
    qes.qes_gaussian_factors(w, w, R, Cs, Sn)
    Ro, Co, So = qo.bm24(words, words)
    for got, want, name in ((R, Ro, "radius"), (Cs, Co, "cos"), (Sn, So, "sin")):
        g = _host(got)
        assert np.array_equal(g.view(np.uint32), want.view(np.uint32)), \
            f"{name}: {(g.view(np.uint32) != want.view(np.uint32)).sum()} of 2^24 values differ"


@pytest.mark.parametrize("name,n_tensors,n_segments", [("decoder7b_int4", 14, 2), ("decoder7b_int8", 7, 1),
                                                       ("decoder8b_int4", 3, 1)])
def test_fused_launch_segments_match_per_tensor_oracle(qo, qes, name, n_tensors, n_segments):
    """The whole-model pass the benchmark times: runs of consecutive tensors go to the library as one
    [numel / 32, 32] tensor (at most 2^28 codes per call).  Checked on the leading tensors of the 7B-shaped INT4
    and INT8 sets and of the 8B-shaped set (N = 64, K = 64) against the oracle run tensor by tensor with each
    tensor's own geometry, on sampled words that include both ends of every tensor."""
    from paper_2602_03120_b200.model_pass import ModelPass, launch_segments
    cfg = wl.WORKLOADS[name]
    tensors = cfg.tensors[:n_tensors]
    model = ModelPass(cfg, tensors=tensors)
    assert len(model.segments) == len(launch_segments(tensors)) == n_segments
    assert sum(t.numel for t, _ in model.segments) == sum(t.numel for t in tensors)
    host = model.host_codes()
    model.load(host)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)
    import torch
    member_seed = int(seeds[-1, 1])
    scratch = torch.empty_like(model.w)
    assert model.perturb_member(scratch, member_seed) == n_segments
    pert_all = _host(scratch)
    assert model.update(_dev(seeds), _dev(fit), cfg.K) == n_segments
    got_all = _host(model.w)
    ho = qo.HParams(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    per_tensor = 512 if cfg.K <= 16 else 128
    near_total = 0
    for ti, t in enumerate(tensors):
        lo, nb = wl.packed_bytes(cfg.bits, t.elem_offset), wl.packed_bytes(cfg.bits, t.numel)
        packed = host[lo:lo + nb]
        assert np.array_equal(packed, wl.draw_codes(cfg, ti))
        to = qo.Tensor(bits=cfg.bits, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
        idx = wl.sample_elements(t.numel, per_tensor, stream=100 + ti)
        ref = qo.update(to, packed, None, seeds, fit, cfg.K, ho, idx=idx)
        got = _codes_at(qo, cfg.bits, got_all[lo:lo + nb], idx)
        near = ref["band"] < BAND
        assert not np.any((got != ref["w_new"]) & ~near), f"tensor {ti} ({t.name})"
        near_total += int(near.sum())
        want_p = qo.perturb(to, packed, None, member_seed, ho, idx=idx)
        assert np.array_equal(_codes_at(qo, cfg.bits, pert_all[lo:lo + nb], idx), want_p), f"tensor {ti} ({t.name}): perturb"
    print(f"fused segments ({name}): near-band sampled elements {near_total}")


@pytest.mark.parametrize("name,n_sample", [("decoder1p5b_int4", 1 << 20), ("decoder7b_int4", 1 << 20),
                                           ("decoder7b_int8", 1 << 20), ("decoder8b_int4", 1 << 17)])
def test_whole_model_through_the_benchmarked_calls(qo, qes, name, n_sample):
    """The full weight set of each large configuration through exactly the calls the benchmark times
    (ModelPass.perturb_member for one member, then ModelPass.update, fused launches of at most 2^28 codes),
    at the configuration's N and K.  The oracle, run tensor by tensor with each tensor's own geometry,
    checks n_sample elements spread over ALL tensors, the first and the last 32-element word of every tensor
    included: perturbed codes bit for bit, updated codes bit for bit outside the counted 1e-5 band."""
    import torch
    from paper_2602_03120_b200.model_pass import ModelPass
    cfg = wl.WORKLOADS[name]
    model = ModelPass(cfg)
    host = model.host_codes()
    model.load(host)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)
    member_seed = int(seeds[-1, cfg.n_pop - 1])
    scratch = torch.empty_like(model.w)
    model.perturb_member(scratch, member_seed)
    pert_all = _host(scratch)
    del scratch
    model.update(_dev(seeds), _dev(fit), cfg.K)
    got_all = _host(model.w)
    ho = qo.HParams(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    per_tensor = max(96, (n_sample // len(cfg.tensors) + 31) // 32 * 32 + 64)
    checked = mismatched = near_total = changed = 0
    for ti, t in enumerate(cfg.tensors):
        lo, nb = wl.packed_bytes(cfg.bits, t.elem_offset), wl.packed_bytes(cfg.bits, t.numel)
        packed = host[lo:lo + nb]
        to = qo.Tensor(bits=cfg.bits, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
        idx = wl.sample_elements(t.numel, per_tensor, stream=500 + ti)
        assert idx[0] == 0 and idx[-1] == t.numel - 1
        ref = qo.update(to, packed, None, seeds, fit, cfg.K, ho, idx=idx)
        got = _codes_at(qo, cfg.bits, got_all[lo:lo + nb], idx)
        near = ref["band"] < BAND
        mismatched += int(((got != ref["w_new"]) & ~near).sum())
        assert np.all(np.abs(got[near] - ref["w_new"][near]) <= 1)
        near_total += int(near.sum())
        changed += int((ref["w_new"] != _codes_at(qo, cfg.bits, packed, idx)).sum())
        want_p = qo.perturb(to, packed, None, member_seed, ho, idx=idx)
        mismatched += int((_codes_at(qo, cfg.bits, pert_all[lo:lo + nb], idx) != want_p).sum())
        checked += idx.size
    print(f"whole model {name}: {checked} elements of {len(cfg.tensors)} tensors checked (update and one perturbed member), "
          f"{mismatched} mismatches, {near_total} inside the rounding band, {changed} changed by the update")
    assert checked >= n_sample and mismatched == 0
    assert near_total < 1e-3 * checked and changed > 0.01 * checked


@pytest.mark.parametrize("bits,off", [(4, (1 << 33) - 1024), (8, (1 << 33) - 32), (4, (1 << 33) - 2048)])
def test_update_where_the_counter_high_word_changes(qo, qes, bits, off):
    """Element 2^33 is where the high word of the Philox counter (pair index >> 32) steps from 0 to 1:
    a tensor that straddles it (inside a thread block, at a block edge, one word before it)."""
    rows, cols, N, K = 12, 512, 5, 2
    to, tg, packed, _ = _case(qo, qes, bits, rows, cols, off=off)
    ho, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=N)
    seeds, fit = wl.draw_seeds(K + 1, N, stream=33), wl.draw_fitness(K + 1, N, stream=33)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), K, None, hg)
    ref = qo.update(to, packed, None, seeds, fit, K, ho)
    _compare_update(qo, _host(w), bits, ref, "counter high word")
    wp = _dev(np.zeros_like(packed))
    qes.qes_perturb(tg, _dev(packed), wp, None, int(seeds[0, 0]), hg)
    assert np.array_equal(_host(wp), qo.pack(bits, qo.perturb(to, packed, None, int(seeds[0, 0]), ho)))


@pytest.mark.parametrize("bits,rows,cols,N,K,sigma,mode,unit", [
    (4, 45, 736, 8, 4, 0.5, 0, 0), (8, 17, 288, 6, 2, 0.5, 1, 0), (4, 9, 512, 4, 3, 2.0, 0, 0), (4, 11, 256, 10, 1, 0.012, 0, 1)])
def test_antithetic_pairs_update_replay_and_perturb(qo, qes, bits, rows, cols, N, K, sigma, mode, unit):
    """App. A's antithetic pairs: N / 2 seeds per generation, fitness interleaved F+, F-; update, history loop
    and the two-member perturbation against the oracle (sigma = 2.0 reaches the symmetric 4-bit limit)."""
    import torch
    group = 128 if (bits == 4 and unit) else 0
    to, tg, packed, scales = _case(qo, qes, bits, rows, cols, group=group, off=32 * 77)
    lr = 2.0 * sigma if unit else 1.0          # weight units: a step of the order of sigma, c = 2 / N
    kw = dict(sigma=sigma, lr=lr, gamma=0.9, n_pop=N, boundary_mode=mode, sigma_unit=unit, antithetic=1)
    ho, hg = _hp(qo, qes, **kw)
    sc_d = _dev(scales) if unit else None
    sc_o = scales if unit else None
    seeds, fit = wl.draw_seeds(K + 1, N // 2, stream=rows), wl.draw_fitness(K + 1, N, stream=rows)
    w = _dev(packed)
    qes.qes_update(tg, w, sc_d, _dev(seeds), _dev(fit), K, None, hg)
    ref = qo.update(to, packed, sc_o, seeds, fit, K, ho)
    _compare_update(qo, _host(w), bits, ref, "antithetic update")
    assert (ref["w_new"] != qo.unpack(bits, packed, rows * cols)).any()
    res = torch.empty(rows * cols, dtype=torch.float32, device="cuda")
    qes.qes_replay_residual(tg, _dev(packed), sc_d, _dev(seeds[:K]), _dev(fit[:K]), K, hg, res)
    rr = qo.replay_residual(to, packed, sc_o, seeds[:K], fit[:K], K, ho)
    far = rr["band"] >= BAND
    assert np.abs(_host(res).astype(np.float64) - rr["e"])[far].max(initial=0.0) <= TOL
    seed = int(seeds[-1, 0])
    wp, wm = _dev(np.zeros_like(packed)), _dev(np.zeros_like(packed))
    qes.qes_perturb_pair(tg, _dev(packed), wp, wm, sc_d, seed, hg)
    assert np.array_equal(_host(wp), qo.pack(bits, qo.perturb(to, packed, sc_o, seed, ho, sign=1)))
    assert np.array_equal(_host(wm), qo.pack(bits, qo.perturb(to, packed, sc_o, seed, ho, sign=-1)))
    one = _dev(np.zeros_like(packed))
    qes.qes_perturb(tg, _dev(packed), one, sc_d, seed, hg)               # the + member alone
    assert np.array_equal(_host(one), _host(wp))
    inplace = _dev(packed)
    qes.qes_perturb_pair(tg, inplace, inplace, wm, sc_d, seed, hg)       # the + output may alias the input
    assert np.array_equal(_host(inplace), _host(wp))


def _half_spacing(x):
    """Spacing of binary16 at |x| (2^-24 in the subnormal range)."""
    a = np.maximum(np.abs(x), 2.0 ** -14)
    return 2.0 ** (np.floor(np.log2(a)) - 10)


def test_stored_residual_in_binary16(qo, qes):
    """Algorithm 1 with the residual kept in FP16: three chained steps, each checked against the oracle started
    from the library's own previous state; codes as usual, the stored residual must be a correct binary16
    rounding of a value within 1e-5 of the oracle's."""
    import torch
    bits, rows, cols, N = 4, 29, 416, 8
    to, tg, packed, _ = _case(qo, qes, bits, rows, cols, off=64)
    n = rows * cols
    kw = dict(sigma=0.5, lr=0.7, gamma=0.9, n_pop=N, residual_f16=1)
    ho, hg = _hp(qo, qes, **kw)
    w = _dev(packed)
    e = torch.zeros(n, dtype=torch.float16, device="cuda")
    for step in range(3):
        w_before, e_before = _host(w).copy(), _host(e).copy()
        seeds, fit = wl.draw_seeds(1, N, stream=200 + step), wl.draw_fitness(1, N, stream=200 + step)
        qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), 0, e, hg)
        ref = qo.update(to, w_before, None, seeds, fit, 0, ho, residual_in=e_before)
        _compare_update(qo, _host(w), bits, ref, f"fp16 residual, step {step}")
        far = ref["band"] >= BAND
        got = _host(e).astype(np.float64)
        assert np.all(np.abs(got - ref["e_new"])[far] <= 0.5 * _half_spacing(ref["e_new"][far]) + TOL)
        assert np.mean(_host(e).view(np.uint16)[far] == qo.to_half(ref["e_new"])[far]) > 0.995
    assert np.any(_host(e) != 0)
    # the history loop can write binary16 too
    K = 3
    seeds, fit = wl.draw_seeds(K, N, stream=210), wl.draw_fitness(K, N, stream=210)
    out = torch.empty(n, dtype=torch.float16, device="cuda")
    qes.qes_replay_residual(tg, _dev(packed), None, _dev(seeds), _dev(fit), K, hg, out)
    rr = qo.replay_residual(to, packed, None, seeds, fit, K, ho)
    far = rr["band"] >= BAND
    assert np.all(np.abs(_host(out).astype(np.float64) - rr["e"])[far] <= 0.5 * _half_spacing(rr["e"][far]) + TOL)


@pytest.mark.parametrize("bits,rows,cols,off,N,K,sigma,mode,anti,unit", [
    (4, 53, 608, 32 * 9, 8, 4, 0.5, 0, 0, 0), (8, 19, 352, (1 << 34) - 1024, 5, 2, 0.5, 1, 0, 0),
    (4, 7, 1024, (1 << 34) - 2048, 6, 3, 2.0, 0, 1, 0), (4, 13, 384, (1 << 41) + 96, 4, 1, 0.012, 0, 0, 1),
    (8, 1, 32, 0, 1, 0, 0.5, 0, 0, 0)])
def test_quad_noise_mode(qo, qes, bits, rows, cols, off, N, K, sigma, mode, anti, unit):
    """noise_mode = QUAD8 (one Philox call per four elements, 8-bit Bernoulli uniforms): perturbation, stateless
    update, history loop and stored residual against the oracle in the same mode, including tensors that
    straddle element 2^34, where the counter high word of this mode changes."""
    import torch
    group = 128 if (bits == 4 and unit) else 0
    to, tg, packed, scales = _case(qo, qes, bits, rows, cols, group=group, off=off)
    lr = 2.0 * sigma if unit else 1.0
    kw = dict(sigma=sigma, lr=lr, gamma=0.9, n_pop=N, boundary_mode=mode, sigma_unit=unit, antithetic=anti, noise_mode=1)
    ho, hg = _hp(qo, qes, **kw)
    sc_d, sc_o = (_dev(scales), scales) if unit else (None, None)
    n_seeds = N // 2 if anti else N
    seeds, fit = wl.draw_seeds(K + 1, n_seeds, stream=300 + rows), wl.draw_fitness(K + 1, N, stream=300 + rows)
    seed = int(seeds[-1, 0])
    wp = _dev(np.zeros_like(packed))
    qes.qes_perturb(tg, _dev(packed), wp, sc_d, seed, hg)
    assert np.array_equal(_host(wp), qo.pack(bits, qo.perturb(to, packed, sc_o, seed, ho)))
    if anti:
        wm = _dev(np.zeros_like(packed))
        qes.qes_perturb_pair(tg, _dev(packed), wp, wm, sc_d, seed, hg)
        assert np.array_equal(_host(wm), qo.pack(bits, qo.perturb(to, packed, sc_o, seed, ho, sign=-1)))
    w = _dev(packed)
    stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    qes.qes_update(tg, w, sc_d, _dev(seeds), _dev(fit), K, None, hg, stats=stats)
    ref = qo.update(to, packed, sc_o, seeds, fit, K, ho)
    n_near = _compare_update(qo, _host(w), bits, ref, "quad noise update")
    assert abs(int(_host(stats)[0]) - int((ref["w_new"] != qo.unpack(bits, packed, rows * cols)).sum())) <= n_near
    plain = qo.update(to, packed, sc_o, seeds, fit, K, qo.HParams(**{**kw, "noise_mode": 0}))
    if rows * cols > 1000:
        assert not np.array_equal(plain["w_new"], ref["w_new"])          # the two modes are different streams
    res = torch.empty(rows * cols, dtype=torch.float32, device="cuda")
    qes.qes_replay_residual(tg, _dev(packed), sc_d, _dev(seeds[:K]), _dev(fit[:K]), K, hg, res)
    rr = qo.replay_residual(to, packed, sc_o, seeds[:K], fit[:K], K, ho)
    far = rr["band"] >= BAND
    assert np.abs(_host(res).astype(np.float64) - rr["e"])[far].max(initial=0.0) <= TOL
    e_in = np.random.default_rng(rows).uniform(-0.5, 0.5, rows * cols).astype(np.float32)
    w2, e2 = _dev(packed), _dev(e_in)
    qes.qes_update(tg, w2, sc_d, _dev(seeds[-1:]), _dev(fit[-1:]), 0, e2, hg)
    ref2 = qo.update(to, packed, sc_o, seeds[-1:], fit[-1:], 0, ho, residual_in=e_in)
    _compare_update(qo, _host(w2), bits, ref2, "quad noise stored residual")
    far2 = ref2["band"] >= BAND
    assert np.abs(_host(e2).astype(np.float64) - ref2["e_new"])[far2].max(initial=0.0) <= TOL


def test_quad_noise_full_size_tensor_sampled(qo, qes):
    """A full-size tensor of the 7B-shaped set in QUAD8 mode at the benchmark's N and K, oracle on sampled words."""
    cfg = wl.WORKLOADS["decoder7b_int4"]
    ti = 6
    t = cfg.tensors[ti]
    kw = dict(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop, noise_mode=1)
    ho, hg = _hp(qo, qes, **kw)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)
    packed = wl.draw_codes(cfg, ti)
    to = qo.Tensor(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
    tg = qes.TensorDesc(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), cfg.K, None, hg)
    idx = wl.sample_elements(t.numel, 2048, stream=77)
    ref = qo.update(to, packed, None, seeds, fit, cfg.K, ho, idx=idx)
    got = qo.unpack(4, _host(w), t.numel)[idx]
    near = ref["band"] < BAND
    assert not np.any((got != ref["w_new"]) & ~near)


@pytest.mark.parametrize("N,anti", [(600, 0), (1066, 0), (2132, 1)])
def test_large_populations_stage_more_than_48_kib(qo, qes, N, anti):
    """Populations whose staged round keys need the opt-in shared-memory size (96 B per seed, two
    generations): 600 seeds = 112.5 KiB, and the documented maximum of 1066 seeds (or pairs)."""
    bits, rows, cols, K = 4, 3, 128, 1
    to, tg, packed, _ = _case(qo, qes, bits, rows, cols, off=96)
    ho, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=N, antithetic=anti)
    n_seeds = N // 2 if anti else N
    seeds, fit = wl.draw_seeds(K + 1, n_seeds, stream=N), wl.draw_fitness(K + 1, N, stream=N)
    w = _dev(packed)
    qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), K, None, hg)
    ref = qo.update(to, packed, None, seeds, fit, K, ho)
    _compare_update(qo, _host(w), bits, ref, f"N = {N}")
    too_many = qes.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=1067 * (2 if anti else 1), antithetic=anti)
    with pytest.raises(qes.QesError):
        qes.qes_update(tg, w, None, _dev(np.zeros(4 * 1067, np.uint64)), _dev(np.zeros(4 * 1067, np.float32)), 1, None, too_many)


def test_model_pass_with_weight_unit_sigma_launches_per_tensor(qo, qes):
    """ModelPass with sigma in weight units: one call per tensor, each with its own group scales."""
    from paper_2602_03120_b200.model_pass import ModelPass
    cfg = wl.WORKLOADS["decoder1p5b_int4"]
    picks = (1, 2)                                         # k_proj, v_proj of layer 0: 256 x 1536 each
    tensors = [cfg.tensors[i] for i in picks]
    model = ModelPass(cfg, tensors=tensors, sigma_unit=qes.SIGMA_WEIGHT)
    model.hp.sigma, model.hp.lr = 0.012, 0.024
    model.scales = [_dev(wl.draw_scales(cfg, i)) for i in picks]
    host = np.concatenate([wl.draw_codes(cfg, i) for i in picks])
    model.load(host)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop)
    assert model.update(_dev(seeds), _dev(fit), cfg.K) == 2
    got = _host(model.w)
    ho = qo.HParams(sigma=0.012, lr=0.024, gamma=cfg.gamma, n_pop=cfg.n_pop, sigma_unit=1)
    lo = 0
    for i in picks:
        t = cfg.tensors[i]
        to = qo.Tensor(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
        idx = wl.sample_elements(t.numel, 4096, stream=i)
        ref = qo.update(to, wl.draw_codes(cfg, i), wl.draw_scales(cfg, i), seeds, fit, cfg.K, ho, idx=idx)
        g = qo.unpack(4, got[lo:lo + t.numel // 2], t.numel)[idx]
        assert not np.any((g != ref["w_new"]) & (ref["band"] >= BAND))
        lo += t.numel // 2


def test_resume_from_weights_and_history_through_the_library(qo, qes):
    """Checkpoint / resume: the optimizer state is the packed weights plus the seed/reward window."""
    from paper_2602_03120_b200.history import SeedHistory
    N, K, T = 6, 3, 6
    tg = qes.TensorDesc(bits=4, rows=16, cols=256)
    hg = qes.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=N)
    w0 = np.random.default_rng(9).integers(0, 256, 2048, dtype=np.uint8)
    gens = [(wl.draw_seeds(1, N, stream=600 + s)[0], wl.draw_fitness(1, N, stream=600 + s)[0]) for s in range(T)]

    def run(w_host, hist, steps):
        w = _dev(w_host)
        for s, f in steps:
            seeds, fit, k = hist.tables(s, f)
            qes.qes_update(tg, w, None, _dev(seeds), _dev(fit), k, None, hg)
            hist.push(s, f)
        return _host(w), hist

    w_full, _ = run(w0, SeedHistory(K, N), gens)
    w_half, hist = run(w0, SeedHistory(K, N), gens[:T // 2])
    w_res, _ = run(np.frombuffer(w_half.tobytes(), np.uint8).copy(), SeedHistory.from_bytes(hist.to_bytes()), gens[T // 2:])
    assert np.array_equal(w_full, w_res) and not np.array_equal(w_full, w0)


def test_random_configurations(qo, qes):
    """Thirty seeded random small cases over every switch of the interface (bit width, ragged shapes, group
    size, element offset, population, window, sigma incl. the 4-bit limit, both units, both boundary rules,
    narrowed code ranges, antithetic pairs, both noise modes): update, history loop and perturbation."""
    import torch
    rng = np.random.default_rng(20260203)
    total_near, report = 0, []
    for case in range(30):
        bits = int(rng.choice([4, 8]))
        rows, cols = int(rng.integers(1, 40)), 32 * int(rng.integers(1, 24))
        unit = int(rng.integers(0, 2))
        group = int(rng.choice([g for g in (0, 32, 64, 128) if g == 0 or cols % g == 0])) if unit else 0
        off = 32 * int(rng.integers(0, 1 << 20)) + (int(rng.integers(0, 4)) << 33)
        anti = int(rng.integers(0, 2))
        N = 2 * int(rng.integers(1, 9)) if anti else int(rng.integers(1, 17))
        K = int(rng.integers(0, 6))
        sigma = float(rng.choice([0.25, 0.5, 1.0, 2.5])) if not unit else float(rng.choice([0.006, 0.012, 0.03]))
        lr = float(rng.choice([0.5, 1.0])) * (2.0 * sigma if unit else 1.0)
        lim = 1 << (bits - 1)
        qmin, qmax = (-lim, lim - 1) if rng.integers(0, 2) else (-(lim - 1) + int(rng.integers(0, 3)), lim - 1 - int(rng.integers(0, 3)))
        kw = dict(sigma=sigma, lr=lr, gamma=float(rng.choice([0.0, 0.9, 1.0])), n_pop=N, sigma_unit=unit,
                  boundary_mode=int(rng.integers(0, 2)), antithetic=anti, noise_mode=int(rng.integers(0, 2)))
        to, tg, packed, scales = _case(qo, qes, bits, rows, cols, group=group, off=off, qmin=qmin, qmax=qmax, seed=case)
        ho, hg = _hp(qo, qes, **kw)
        sc_d, sc_o = (_dev(scales), scales) if unit else (None, None)
        seeds = wl.draw_seeds(K + 1, N // 2 if anti else N, stream=1000 + case)
        fit = wl.draw_fitness(K + 1, N, "student_t3" if case % 3 == 0 else "normal", stream=1000 + case)
        what = f"case {case}: bits {bits} {rows}x{cols} g{group} N{N} K{K} {kw}"
        w = _dev(packed)
        qes.qes_update(tg, w, sc_d, _dev(seeds), _dev(fit), K, None, hg)
        ref = qo.update(to, packed, sc_o, seeds, fit, K, ho)
        total_near += _compare_update(qo, _host(w), bits, ref, what)
        got = qo.unpack(bits, _host(w), rows * cols)
        assert got.min() >= qmin and got.max() <= qmax, what
        res = torch.empty(rows * cols, dtype=torch.float32, device="cuda")
        qes.qes_replay_residual(tg, _dev(packed), sc_d, _dev(seeds[:K]), _dev(fit[:K]), K, hg, res)
        rr = qo.replay_residual(to, packed, sc_o, seeds[:K], fit[:K], K, ho)
        far = rr["band"] >= BAND
        worst = float(np.abs(_host(res).astype(np.float64) - rr["e"])[far].max(initial=0.0))
        report.append((case, float(np.abs(rr["e"]).max(initial=0.0)), worst))
        assert worst <= TOL, what
        seed = int(seeds[-1, 0])
        wp = _dev(np.zeros_like(packed))
        qes.qes_perturb(tg, _dev(packed), wp, sc_d, seed, hg)
        assert np.array_equal(_host(wp), qo.pack(bits, qo.perturb(to, packed, sc_o, seed, ho))), what
    print(f"random configurations: {total_near} elements inside the rounding band; residual error per case "
          f"(case, max |e|, max |e_gpu - e_oracle|): " + ", ".join(f"({c}, {m:.3g}, {w:.2g})" for c, m, w in report))


def test_step_from_host_equals_the_resident_step(qo, qes):
    """The end-to-end call (weights in pinned host memory, copies pipelined under the arithmetic on side
    streams) gives the bytes of the resident path, twice in a row, and leaves the last member's perturbation
    in the scratch copy."""
    import torch
    from paper_2602_03120_b200.model_pass import ModelPass, MAX_SEGMENT_ELEMS
    cfg = wl.WORKLOADS["decoder1p5b_int4"]
    tensors = cfg.tensors[:14]                                   # two layers, 93.6M codes
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop), wl.draw_fitness(cfg.K + 1, cfg.n_pop)
    member_seeds = [int(s) for s in seeds[-1][:3]]
    import paper_2602_03120_b200.model_pass as mp
    old = mp.MAX_SEGMENT_ELEMS
    mp.MAX_SEGMENT_ELEMS = 1 << 25                               # several launches, so the pipeline has stages
    try:
        model = ModelPass(cfg, tensors=tensors)
        segs = mp.launch_segments(tensors, mp.MAX_SEGMENT_ELEMS)
        model.segments = [(wl.TensorSpec(f"segment{j}", n // 32, 32, off),
                           qes.TensorDesc(bits=4, rows=n // 32, cols=32, elem_offset=off)) for j, (_, off, n) in enumerate(segs)]
        assert len(model.segments) >= 3
    finally:
        mp.MAX_SEGMENT_ELEMS = old
    host = torch.from_numpy(model.host_codes()).pin_memory()
    out = torch.empty_like(host).pin_memory()
    scratch = torch.empty_like(model.w)
    ds, df = _dev(seeds), _dev(fit)
    model.load(host)
    model.update(ds, df, cfg.K)
    want = _host(model.w)
    want_scratch = torch.empty_like(model.w)
    model.load(host)
    model.perturb_member(want_scratch, member_seeds[-1])
    for _ in range(2):
        out.zero_()
        n = model.step_from_host(host, out, scratch, member_seeds, ds, df, cfg.K)
        torch.cuda.synchronize()
        assert n == len(model.segments) * (len(member_seeds) + 1)
        assert np.array_equal(out.numpy(), want)
        assert torch.equal(scratch, want_scratch)
    assert not np.array_equal(want, host.numpy())


def test_calls_run_on_the_callers_stream(qo, qes):
    """The library enqueues on the stream it is given and returns without synchronising.  The side stream is kept
    busy first and the weights are only copied into place at the end of ITS queue: a kernel launched anywhere else
    (torch's side streams do not synchronise with the default stream) would run before the copy and its result be
    overwritten; and an event recorded on the side stream right after the call is still pending when the call
    returns."""
    import torch
    to, tg, packed, _ = _case(qo, qes, 4, 64, 512, off=128)
    _, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=8)
    seeds, fit = _dev(wl.draw_seeds(4, 8, stream=7)), _dev(wl.draw_fitness(4, 8, stream=7))
    want = _dev(packed)
    qes.qes_update(tg, want, None, seeds, fit, 3, None, hg)
    src = _dev(packed)
    torch.cuda.synchronize()
    for explicit in (True, False):
        s1 = torch.cuda.Stream()
        w = torch.zeros_like(src)
        torch.cuda.synchronize()
        with torch.cuda.stream(s1):
            torch.cuda._sleep(400_000_000)                      # roughly 0.2 s of the side stream's time
            w.copy_(src, non_blocking=True)
            if not explicit:
                qes.qes_update(tg, w, None, seeds, fit, 3, None, hg)     # the stream comes from torch's current stream
        if explicit:
            qes.qes_update(tg, w, None, seeds, fit, 3, None, hg, stream=s1)   # the stream is passed, another one is current
        done = torch.cuda.Event(); done.record(s1)
        assert not done.query(), "the call waited for the stream"
        s1.synchronize()
        assert torch.equal(w, want)


def test_weight_unit_sigma_with_extreme_scales(qo, qes):
    """sigma in weight units over scales at the ends of binary16: zero (sigma / 0 = +inf acts as 2^40: every
    non-zero sample saturates the 4-bit range, a zero sample stays zero), the smallest subnormal, the largest finite
    value, and an ordinary one -- perturbation bit for bit, update and history loop within the usual rules."""
    import torch
    rows, cols, N, K = 8, 256, 6, 2
    for bits, group in ((4, 64), (8, 0)):
        to, tg, packed, _ = _case(qo, qes, bits, rows, cols, group=group, off=32 * 11)
        n_scales = rows * (cols // group) if group else rows
        scales = np.resize(np.array([0.0, 2.0 ** -24, 65504.0, 0.0125], np.float16), n_scales)
        for sigma in (0.02, 1e29):
            kw = dict(sigma=sigma, lr=2.0 * sigma, gamma=0.9, n_pop=N, sigma_unit=1)
            ho, hg = _hp(qo, qes, **kw)
            seeds, fit = wl.draw_seeds(K + 1, N, stream=91), wl.draw_fitness(K + 1, N, stream=91)
            wp = _dev(np.zeros_like(packed))
            qes.qes_perturb(tg, _dev(packed), wp, _dev(scales), int(seeds[0, 0]), hg)
            assert np.array_equal(_host(wp), qo.pack(bits, qo.perturb(to, packed, scales, int(seeds[0, 0]), ho)))
            w = _dev(packed)
            qes.qes_update(tg, w, _dev(scales), _dev(seeds), _dev(fit), K, None, hg)
            ref = qo.update(to, packed, scales, seeds, fit, K, ho)
            _compare_update(qo, _host(w), bits, ref, f"extreme scales, sigma {sigma}")
            res = torch.empty(rows * cols, dtype=torch.float32, device="cuda")
            qes.qes_replay_residual(tg, _dev(packed), _dev(scales), _dev(seeds[:K]), _dev(fit[:K]), K, hg, res)
            rr = qo.replay_residual(to, packed, scales, seeds[:K], fit[:K], K, ho)
            far = rr["band"] >= BAND
            assert np.abs(_host(res).astype(np.float64) - rr["e"])[far].max(initial=0.0) <= TOL


def test_tensor_with_more_than_2_pow_32_codes(qo, qes):
    """One INT4 tensor of 2^32 + 2^20 codes (2 GiB packed): element and chunk indices pass 32 bits inside a single
    launch.  Perturbation and a small stateless update, checked on sampled words that include the last ones."""
    import torch
    rows, cols = (1 << 17) + 32, 1 << 15
    n = rows * cols
    assert n > (1 << 32)
    off = 32 * 5
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    w0 = torch.randint(0, 256, (n // 2,), dtype=torch.uint8, device="cuda", generator=g)
    idx = np.unique(np.concatenate([wl.sample_elements(n, 4096, stream=321),
                                    (np.arange(64)[:, None] * 32 + np.arange(32)[None, :]).reshape(-1) + ((1 << 32) - 1024)]))
    words = idx.reshape(-1, 32)[:, 0] // 32
    assert idx[-1] == n - 1 and (idx > (1 << 32)).sum() > 1000
    widx = torch.from_numpy(words).cuda()
    before = w0.view(-1, 16)[widx].cpu().numpy()
    sparse = np.zeros(n // 2, np.uint8)                       # untouched pages cost nothing
    sparse.reshape(-1, 16)[words] = before
    to = qo.Tensor(bits=4, rows=rows, cols=cols, elem_offset=off)
    tg = qes.TensorDesc(bits=4, rows=rows, cols=cols, elem_offset=off)
    N, K = 2, 1
    ho, hg = _hp(qo, qes, sigma=0.5, lr=1.0, gamma=0.9, n_pop=N)
    seeds, fit = wl.draw_seeds(K + 1, N, stream=322), wl.draw_fitness(K + 1, N, stream=322)
    out = torch.empty_like(w0)
    qes.qes_perturb(tg, w0, out, None, int(seeds[0, 0]), hg)
    got_p = qo.unpack(4, out.view(-1, 16)[widx].cpu().numpy().reshape(-1), idx.size)
    assert np.array_equal(got_p, qo.perturb(to, sparse, None, int(seeds[0, 0]), ho, idx=idx))
    del out
    qes.qes_update(tg, w0, None, _dev(seeds), _dev(fit), K, None, hg)
    ref = qo.update(to, sparse, None, seeds, fit, K, ho, idx=idx)
    got = qo.unpack(4, w0.view(-1, 16)[widx].cpu().numpy().reshape(-1), idx.size)
    near = ref["band"] < BAND
    assert not np.any((got != ref["w_new"]) & ~near)
    assert (got != qo.unpack(4, before.reshape(-1), idx.size)).any()
