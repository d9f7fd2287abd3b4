#!/usr/bin/env python
"""Benchmark of the QES parameter pass: one "step" = the whole hot path over one weight set
(qes_perturb for every population member, then the stateless qes_update with seed replay).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is weights updated per second over all ranks with inputs
resident in HBM; `e2e` is the same metric with the weights starting and ending in pinned host
memory (host<->device copies inside the timed region); `roofline` is the fused update kernel
against the SM issue peak (the path is bound by integer/fp32 arithmetic, not by HBM);
`cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload; `parity` compares
sampled elements of one untimed step's output with that oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_03120_b200 import workloads as wl  # noqa: E402

# Algorithmic operation counts of the noise contract (one count per 32-bit multiply, xor, add,
# shift, conversion, compare/select or fp32 operation the definition requires; square root = 1):
#   per Philox call (two samples): 10 rounds x (2 wide multiplies + 2 three-input xors)      = 40
#   Box-Muller pair: radius 20 (uniform 3, log 16, sqrt 1), angle 19 (reduction 7, two
#                    polynomials 8, quadrant 4), sigma scaling 3                              = 42
#   Eq. 3 + Eq. 5 per sample: floor, fraction, shift, compare, add, weighted fma = 7 (x2)    = 14
OPS_PER_SAMPLE = (40 + 42 + 14) / 2.0
# quad8: one Philox call (40) and two Box-Muller pairs (2 x 42) serve four samples (4 x 7)
OPS_PER_SAMPLE_QUAD8 = (40 + 2 * 42 + 4 * 7) / 4.0
OPS_PER_ELEM_GEN = 8.0      # u (2), round, w + step, two compares, select, residual
OPS_PER_ELEM = 6.0          # unpack / repack
SM_COUNT, LANES_PER_SM = 148, 128
# DRAM bytes of one update launch per algorithmic byte (packed weights read once and written once), from the
# ncu capture of this kernel summarised in profiles/pass_kernel_int4_decoder1p5b_segment.md (below 1: part of
# the last writes is still in the 126 MB L2 when the kernel ends).  None = the kernel has changed since the
# counters were taken.
DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE = 0.80
TRAFFIC_SOURCE = "scaled by codes from the one-launch ncu capture in profiles/pass_kernel_int4_decoder1p5b_segment.md"

# Per-pipe form of the same roofline (default noise mode).  Scheduler cycles one warp instruction holds its pipe,
# measured with qes_pipe_probe (profiles/pipe_probes_b200.md), and the instructions per noise sample that the
# kernel's own path -- special-function estimate, verification, weighted sum -- needs on each pipe
# (per Philox call = two samples: 20 wide multiplies and 20 xor3 by the definition of Philox4x32-10; fp32:
# two multiplies each for radius and angle, the sigma scaling, two biased products, two offset removals, two
# weighted-sum fmas = 11; integer pipe besides the xor3: uniform and angle conversions 3, two shift-adds,
# two verifications, one radius-limit test, two top-byte additions = 10; special-function unit: lg2, sqrt,
# sin, cos and the two floors = 6).
PIPE_CYCLES = {"multiply_fp32": {"wide_multiply": 4.02, "fp32": 1.03}, "integer": {"int": 2.01}, "special_function": {"sfu": 8.0}}
PIPE_OPS_PER_SAMPLE = {"multiply_fp32": {"wide_multiply": 10.0, "fp32": 5.5}, "integer": {"int": 15.0}, "special_function": {"sfu": 3.0}}


def pipe_roofline(cycles_per_warp_sample: float):
    """Each pipe's busy cycles per (warp, sample) at the measured rates, as a share of the measured cycles."""
    pipes = {}
    for pipe, kinds in PIPE_OPS_PER_SAMPLE.items():
        busy = sum(n * PIPE_CYCLES[pipe][k] for k, n in kinds.items())
        pipes[pipe] = {"ops_per_sample": sum(kinds.values()), "cycles_per_warp_sample": busy,
                       "time_frac": busy / cycles_per_warp_sample}
    return pipes


def alu_ops(numel: int, n_pop: int, generations: int, per_sample: float = OPS_PER_SAMPLE) -> float:
    return numel * (n_pop * generations * per_sample + generations * OPS_PER_ELEM_GEN + OPS_PER_ELEM)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d.get("hbm_gbs", 6650.0)), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        clk = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i] == "Active" for r in self.rows)]
        pw = [float(r[2]) for r in self.rows if len(r) >= 7 and r[2].replace(".", "").isdigit()]
        return {"sm_mhz": float(np.median(clk)) if clk else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(clk), "reasons": reasons}


def sample_words(cfg: wl.Workload, n_words: int, stream: int) -> np.ndarray:
    """Sorted ids of 32-element words of the flat weight set: the first and the last word of every tensor
    plus words drawn uniformly over the whole set."""
    rng = np.random.default_rng([wl.MASTER_SEED, 6, stream])
    ends = np.array([[t.elem_offset // 32, (t.elem_offset + t.numel) // 32 - 1] for t in cfg.tensors]).reshape(-1)
    extra = rng.integers(0, cfg.numel // 32, size=max(0, n_words - ends.size))
    return np.unique(np.concatenate([ends, extra])).astype(np.int64)


def flat_oracle_tensor(qo, cfg: wl.Workload):
    """The whole weight set as one [numel / 32, 32] tensor: with sigma in grid units the noise depends on the
    global element index alone, so this is the same computation as tensor by tensor."""
    return qo.Tensor(bits=cfg.bits, rows=cfg.numel // 32, cols=32, group_size=0, elem_offset=cfg.tensors[0].elem_offset)


def sparse_packed(cfg: wl.Workload, words: np.ndarray, word_bytes: np.ndarray) -> np.ndarray:
    """A packed buffer of the whole set that holds `word_bytes` at the sampled words (untouched pages cost nothing)."""
    per_word = 32 if cfg.bits == 8 else 16
    buf = np.zeros(wl.packed_bytes(cfg.bits, cfg.numel), np.uint8)
    buf.reshape(-1, per_word)[words] = word_bytes.reshape(-1, per_word)
    return buf


def oracle_rate(cfg: wl.Workload, target_seconds: float = 15.0, antithetic: bool = False, quad: bool = False):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload: whole 32-element words -- the
    first and last word of every tensor plus words drawn uniformly over the set -- holding uniform random
    codes, one full step on them (the perturbation of every member, then the stateless update) at the
    configuration's N and K.  Returns a dict."""
    from oracle import qes_oracle as qo
    qo.build()
    threads = qo.default_threads()
    n_seeds = cfg.n_pop // 2 if antithetic else cfg.n_pop
    seeds, fit = wl.draw_seeds(cfg.K + 1, n_seeds), wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)
    to = flat_oracle_tensor(qo, cfg)
    hp = qo.HParams(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop, antithetic=int(antithetic),
                    noise_mode=int(quad))
    per_elem = n_seeds * (cfg.K + 1)
    per_word = 32 if cfg.bits == 8 else 16

    def one_step(n_words, stream):
        words = sample_words(cfg, n_words, stream)
        codes = np.random.default_rng([wl.MASTER_SEED, 7, stream]).integers(0, 256, size=words.size * per_word, dtype=np.uint8)
        packed = sparse_packed(cfg, words, codes)
        idx = (words[:, None] * 32 + np.arange(32)[None, :]).reshape(-1)
        t0 = time.perf_counter()
        for s in seeds[-1]:                                           # Algorithm 1, member loop
            qo.perturb(to, packed, None, int(s), hp, idx=idx)
            if antithetic:
                qo.perturb(to, packed, None, int(s), hp, idx=idx, sign=-1)
        qo.update(to, packed, None, seeds, fit, cfg.K, hp, idx=idx)   # Algorithm 2
        return idx.size, time.perf_counter() - t0

    n_ends = 2 * len(cfg.tensors)
    n0, dt0 = one_step(max(n_ends, 1024), 900)                        # sizing probe
    n_words = int(max(n_ends, min(cfg.numel // 32, (n0 / dt0) * target_seconds / 32)))
    n, dt = one_step(n_words, 901)
    return {"weights_per_s": n / dt, "samples_per_s": n * per_elem / dt, "cores": threads,
            "elements": int(n), "seconds": dt}


def parity_check(qo_mod, cfg: wl.Workload, before: np.ndarray, after: np.ndarray, perturbed: np.ndarray,
                 words: np.ndarray, seeds, fit, member_seed: int, antithetic: bool, quad: bool):
    """Sampled words of one step's output against the oracle: the updated codes (bit-exact outside the counted
    1e-5 rounding band) and the last member's perturbed copy (bit-exact)."""
    qo = qo_mod
    to = flat_oracle_tensor(qo, cfg)
    hp = qo.HParams(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop, antithetic=int(antithetic), noise_mode=int(quad))
    idx = (words[:, None] * 32 + np.arange(32)[None, :]).reshape(-1)
    packed = sparse_packed(cfg, words, before)
    ref = qo.update(to, packed, None, seeds, fit, cfg.K, hp, idx=idx)
    near = ref["band"] < 1e-5
    got = qo.unpack(cfg.bits, after, idx.size)
    want_p = qo.perturb(to, packed, None, member_seed, hp, idx=idx)
    got_p = qo.unpack(cfg.bits, perturbed, idx.size)
    return {"checked": int(idx.size), "mismatch": int(((got != ref["w_new"]) & ~near).sum()), "near_band": int(near.sum()),
            "perturb_checked": int(idx.size), "perturb_mismatch": int((got_p != want_p).sum()),
            "changed": int((ref["w_new"] != qo.unpack(cfg.bits, before, idx.size)).sum()),
            "sample": "first and last 32-element word of every tensor plus uniformly drawn words; one untimed step "
                      "(last member's perturbed copy, then the stateless update) against the CPU oracle"}


def run_reference(args, cfg):
    """--impl reference: the oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = max(1.0, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    rates = [oracle_rate(cfg, per_step, args.antithetic, args.noise_mode == "quad8") for _ in range(args.warmup + args.steps)][args.warmup:]
    tot_w = sum(r["elements"] for r in rates); tot_t = sum(r["seconds"] for r in rates)
    value = tot_w / tot_t
    line = {"impl": "reference", "metric": "weights_updated_per_s", "value": value, "unit": "weights/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / len(rates),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int4+f32" if cfg.bits == 4 else "int8+f32",
            "data": "synthetic", "config": config_dict(cfg, args.gpus, args.antithetic, args.noise_mode),
            "noise_samples_per_s": value * cfg.n_pop * (cfg.K + 1),
            "cpu_baseline": {"value": value, "unit": "weights/s", "cores": rates[0]["cores"], "kind": "oracle",
                             "sample": f"{rates[0]['elements']} elements per step (first and last 32-element word of every tensor "
                                       f"plus uniformly drawn words), one full step (perturb x N, update), N={cfg.n_pop}, K={cfg.K}"},
            "e2e": {"value": value, "unit": "weights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(cfg, n_gpus, antithetic=False, noise_mode="pair24"):
    return {"population": "antithetic pairs" if antithetic else "independent members", "noise_mode": noise_mode, "workload": cfg.name, "bits": cfg.bits, "weights_per_gpu": cfg.numel, "tensors_per_gpu": len(cfg.tensors),
            "n_pop": cfg.n_pop, "K": cfg.K, "sigma": cfg.sigma, "lr": cfg.lr, "gamma": cfg.gamma,
            "sigma_unit": "grid", "boundary": "gate", "perturb_members_per_step": cfg.n_pop,
            "launches": "one library call per run of consecutive tensors, at most 2^28 codes each",
            "parallelism": f"{n_gpus} x independent shards (no collective)",
            "l2": "weight set (>= 655 MB for the decoder sets) far exceeds the 126 MB L2; "
                  "the 8 MB single-matrix set is flushed by a 256 MB write between steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="decoder7b_int4", choices=list(wl.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--antithetic", action="store_true",
                    help="the population is N/2 antithetic pairs (App. A): N/2 seeds per generation, both members of a "
                         "pair perturbed from one noise pass")
    ap.add_argument("--noise-mode", default="pair24", choices=["pair24", "quad8"],
                    help="pair24 (default): one Philox call per two elements, 24-bit Bernoulli uniforms; quad8: one call "
                         "per four elements, 8-bit Bernoulli uniforms")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
    args = ap.parse_args()
    cfg = wl.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2602_03120_b200 import binding as qes
    from paper_2602_03120_b200.model_pass import ModelPass

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the parameter pass has no CPU path")
    qes.load()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    quad = args.noise_mode == "quad8"
    model = ModelPass(cfg, rank=rank, world=world, antithetic=args.antithetic, noise_mode=int(quad))
    n_seeds = cfg.n_pop // 2 if args.antithetic else cfg.n_pop
    host = torch.from_numpy(model.host_codes()).pin_memory()
    host_out = torch.empty_like(host).pin_memory()
    model.load(host)
    seeds_h = torch.from_numpy(wl.draw_seeds(cfg.K + 1, n_seeds).view(np.int64)).pin_memory()
    fit_h = torch.from_numpy(wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist)).pin_memory()
    seeds, fit = seeds_h.cuda(), fit_h.cuda()
    member_seeds = [int(s) for s in wl.draw_seeds(cfg.K + 1, n_seeds)[-1]]
    scratch = torch.empty_like(model.w)
    scratch_minus = torch.empty_like(model.w) if args.antithetic else None

    def perturb_all():
        n = 0
        for s in member_seeds:                                  # Algorithm 1, member loop
            n += model.perturb_pair(scratch, scratch_minus, s) if args.antithetic else model.perturb_member(scratch, s)
        return n

    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if model.bytes < (512 << 20) else None
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(timers=None):
        launches = 0
        if flush is not None:
            flush.fill_(1)
        if timers is not None:
            a, b, c = ev(), ev(), ev(); a.record(stream)
        launches += perturb_all()
        if timers is not None:
            b.record(stream)
        n_upd = model.update(seeds, fit, cfg.K)                 # Algorithm 2
        if timers is not None:
            c.record(stream); timers.append((a, b, c))
        return launches + n_upd, n_upd

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local); sampler.start()
    timers, launches, n_upd_launches = [], 0, 0
    t_begin, t_end = ev(), ev()
    t_begin.record(stream)
    for _ in range(args.steps):
        n_all, n_upd = step(timers)
        launches += n_all; n_upd_launches += n_upd
    t_end.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = t_begin.elapsed_time(t_end)
    perturb_ms = sum(a.elapsed_time(b) for a, b, _ in timers)
    update_ms = sum(b.elapsed_time(c) for _, b, c in timers)
    if world > 1:
        t = torch.tensor([total_ms, perturb_ms, update_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, perturb_ms, update_ms = t.tolist()
    ms_per_step = total_ms / args.steps
    value = world * model.numel / (ms_per_step * 1e-3)

    # end to end: weights start and end in pinned host memory
    e2e = None
    if not args.no_e2e:
        e2e_steps = args.steps
        barrier()
        a, b = ev(), ev(); a.record(stream)
        for _ in range(e2e_steps):
            s_d, f_d = seeds_h.cuda(non_blocking=True), fit_h.cuda(non_blocking=True)
            model.step_from_host(host, host_out, scratch, member_seeds, s_d, f_d, cfg.K, scratch_minus)
        b.record(stream)
        barrier()
        e_ms = a.elapsed_time(b) / e2e_steps
        if world > 1:
            t = torch.tensor([e_ms], device="cuda", dtype=torch.float64); dist.all_reduce(t, op=dist.ReduceOp.MAX); e_ms = t.item()
        e2e = {"value": world * model.numel / (e_ms * 1e-3), "unit": "weights/s",
               "h2d_bytes_per_step": int(host.numel() + seeds_h.numel() * 8 + fit_h.numel() * 4),
               "d2h_bytes_per_step": int(host_out.numel()), "steps": e2e_steps, "ms_per_step": e_ms}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # parity of one more (untimed) step against the CPU oracle, on sampled words of the whole set
    parity = None
    if not args.no_parity and world == 1:
        from oracle import qes_oracle as qo
        qo.build()
        per_word = 32 if cfg.bits == 8 else 16
        words = sample_words(cfg, 2048 + 2 * len(cfg.tensors), stream=950)
        widx = torch.from_numpy(words).cuda()
        before = model.w.view(-1, per_word)[widx].cpu().numpy().reshape(-1)
        step()
        torch.cuda.synchronize()
        after = model.w.view(-1, per_word)[widx].cpu().numpy().reshape(-1)
        pert = scratch.view(-1, per_word)[widx].cpu().numpy().reshape(-1)
        parity = parity_check(qo, cfg, before, after, pert, words, wl.draw_seeds(cfg.K + 1, n_seeds),
                              wl.draw_fitness(cfg.K + 1, cfg.n_pop, cfg.reward_dist), member_seeds[-1], args.antithetic, quad)

    hbm_gbs, sm_mhz, peak_src = measured_peaks()
    G = cfg.K + 1
    per_sample = OPS_PER_SAMPLE_QUAD8 if quad else OPS_PER_SAMPLE
    upd_ops_per_launch = alu_ops(model.numel, n_seeds, G, per_sample) * args.steps / n_upd_launches
    upd_s_per_launch = update_ms * 1e-3 / n_upd_launches
    alu_peak = SM_COUNT * LANES_PER_SM * sm_mhz * 1e6
    achieved = upd_ops_per_launch / upd_s_per_launch
    bytes_per_launch = 2 * wl.packed_bytes(cfg.bits, model.numel) * args.steps / n_upd_launches
    # the capture was taken on the INT4 kernel in the default noise mode with independent members: other kernels get no figure
    traffic = None if (DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE is None or quad or args.antithetic or cfg.bits != 4) else DRAM_TRAFFIC_PER_ALGORITHMIC_BYTE * bytes_per_launch
    # scheduler cycles per (warp, sample): launch time x clock x schedulers / warp-samples of the launch
    warp_samples = model.numel * n_seeds * G * args.steps / n_upd_launches / 32.0
    cycles_per_warp_sample = upd_s_per_launch * sm_mhz * 1e6 * SM_COUNT * 4 / warp_samples
    pipes = None if quad else pipe_roofline(cycles_per_warp_sample)
    roofline = {"bound": "alu", "kernel": f"pass_kernel<{cfg.bits}> (qes_update, stateless)",
                "achieved": achieved / 1e9, "peak": alu_peak / 1e9, "unit": "Glane-op/s", "frac": achieved / alu_peak,
                "peak_source": f"{SM_COUNT} SMs x 4 schedulers x 32 lanes x {sm_mhz:.0f} MHz (one instruction per scheduler "
                               f"per cycle; SM clock from the {peak_src} peaks file)",
                "ops_per_sample": per_sample, "avg_launch_ms": upd_s_per_launch * 1e3, "launches": n_upd_launches,
                "traffic": traffic, "traffic_source": TRAFFIC_SOURCE if traffic is not None else None,
                "cycles_per_warp_sample": cycles_per_warp_sample, "pipes": pipes,
                "frac_pipe": None if pipes is None else max(v["time_frac"] for v in pipes.values()),
                "pipe_source": "instruction mix of the kernel's own path per sample x cycles per warp instruction measured by "
                               "qes_pipe_probe (profiles/pipe_probes_b200.md)",
                "hbm": {"achieved_gbs": bytes_per_launch / upd_s_per_launch / 1e9, "peak_gbs": hbm_gbs,
                        "frac": bytes_per_launch / upd_s_per_launch / 1e9 / hbm_gbs, "of": peak_src}}
    line = {"metric": "weights_updated_per_s", "value": value, "unit": "weights/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int4+f32" if cfg.bits == 4 else "int8+f32",
            "data": "synthetic", "config": config_dict(cfg, world, args.antithetic, args.noise_mode),
            "noise_samples_per_s": world * model.numel * n_seeds * G / (update_ms * 1e-3 / args.steps),
            "update_ms_per_step": update_ms / args.steps, "perturb_ms_per_step": perturb_ms / args.steps,
            "perturb_weights_per_s": world * model.numel * cfg.n_pop / (perturb_ms * 1e-3 / args.steps),
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "e2e": e2e, "parity": parity}
    if not args.no_cpu_baseline and world == 1:
        r = oracle_rate(cfg, antithetic=args.antithetic, quad=quad)
        line["cpu_baseline"] = {"value": r["weights_per_s"], "unit": "weights/s", "cores": r["cores"], "kind": "oracle",
                                "samples_per_s": r["samples_per_s"],
                                "sample": f"{r['elements']} elements (first and last 32-element word of every tensor plus uniformly "
                                          f"drawn words), one full step (perturb x N, update), N={cfg.n_pop}, K={cfg.K}, {r['seconds']:.1f} s"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
