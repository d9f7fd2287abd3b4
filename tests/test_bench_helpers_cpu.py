"""The benchmark's own parity accounting, checked on the CPU: the flat [numel / 32, 32] view of a weight set gives
the oracle's per-tensor results, sampled words include both ends of every tensor, a correct output counts zero
mismatches and a planted wrong code is counted."""
import numpy as np

import bench
from paper_2602_03120_b200 import workloads as wl


def _tiny():
    return wl._make("tiny_int4", 4, 64, 4, 2, 2, (("a", 8, 128), ("b", 4, 64), ("c", 16, 256)))


def test_sample_words_cover_both_ends_of_every_tensor():
    cfg = _tiny()
    words = bench.sample_words(cfg, 40, stream=1)
    assert np.all(np.diff(words) > 0)
    for t in cfg.tensors:
        assert t.elem_offset // 32 in words and (t.elem_offset + t.numel) // 32 - 1 in words
    assert words.min() >= 0 and words.max() == cfg.numel // 32 - 1


def test_parity_check_counts_zero_on_the_oracles_output_and_one_on_a_planted_error(qo):
    cfg = _tiny()
    rng = np.random.default_rng(0)
    full = rng.integers(0, 256, cfg.numel // 2, dtype=np.uint8)
    seeds, fit = wl.draw_seeds(cfg.K + 1, cfg.n_pop, stream=3), wl.draw_fitness(cfg.K + 1, cfg.n_pop, stream=3)
    hp = qo.HParams(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    member_seed = int(seeds[-1, -1])
    # the expected output, tensor by tensor with each tensor's own geometry
    upd, pert = np.empty(cfg.numel, np.int32), np.empty(cfg.numel, np.int32)
    for t in cfg.tensors:
        lo = t.elem_offset
        to = qo.Tensor(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=lo)
        packed = full[lo // 2:(lo + t.numel) // 2]
        upd[lo:lo + t.numel] = qo.update(to, packed, None, seeds, fit, cfg.K, hp)["w_new"]
        pert[lo:lo + t.numel] = qo.perturb(to, packed, None, member_seed, hp)
    words = bench.sample_words(cfg, 30, stream=2)
    take = lambda packed: packed.reshape(-1, 16)[words].reshape(-1)
    after, perturbed = qo.pack(4, upd), qo.pack(4, pert)
    r = bench.parity_check(qo, cfg, take(full), take(after), take(perturbed), words, seeds, fit, member_seed, False, False)
    assert r["checked"] == words.size * 32 and r["mismatch"] == 0 and r["perturb_mismatch"] == 0 and r["changed"] > 0
    # plant one wrong updated code (far from any rounding band: move it by 3) and one wrong perturbed code
    bad = take(after).copy(); bad[5] ^= 0x03
    badp = take(perturbed).copy(); badp[-1] ^= 0x30
    r = bench.parity_check(qo, cfg, take(full), bad, badp, words, seeds, fit, member_seed, False, False)
    assert r["mismatch"] + (1 if r["near_band"] else 0) >= 1 and r["perturb_mismatch"] == 1


def test_pipe_roofline_shares():
    pipes = bench.pipe_roofline(60.0)
    assert set(pipes) == {"multiply_fp32", "integer", "special_function"}
    assert abs(pipes["multiply_fp32"]["cycles_per_warp_sample"] - (10 * 4.02 + 5.5 * 1.03)) < 1e-9
    assert max(p["time_frac"] for p in pipes.values()) == pipes["multiply_fp32"]["time_frac"] < 1.0
