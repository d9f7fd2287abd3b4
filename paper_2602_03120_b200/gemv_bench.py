"""Times the batch-1 weight read of a decoder-shaped INT4 set, plain and with the member's perturbation generated in
the read (``python -m paper_2602_03120_b200.gemv_bench [--workload decoder7b_int4]``).

One "read" is one decode step's pass over every linear layer's packed weights (qes_gemv per tensor).  Per layer
shape the tensors of all layers are read back to back, so every launch reads weights that are not in L2 (the
k/v projections are the exception: all their copies together are smaller than L2, which the table says).  Each
pass is captured in a CUDA graph and replayed (the kernels are shorter than a host call), timed with CUDA events
after three warm-up passes, mean of the replays; bandwidth counts the packed codes and scales read once.  The last column is qes_perturb writing a stored copy of the same tensors, for scale.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding as qes
from . import workloads as wl

L2_BYTES = 126 << 20


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="decoder7b_int4", choices=[n for n, w in wl.WORKLOADS.items() if w.bits == 4])
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("gemv_bench needs a CUDA device")
    qes.load()
    cfg = wl.WORKLOADS[args.workload]
    peaks = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    hbm = json.load(open(peaks))["hbm_gbs"] if os.path.exists(peaks) else 6650.0
    peak_src = "measured" if os.path.exists(peaks) else "fallback"
    rng = np.random.default_rng([wl.MASTER_SEED, 8])
    w = torch.from_numpy(rng.integers(0, 256, cfg.numel // 2, dtype=np.uint8)).cuda()      # uniform random codes
    scratch = torch.empty_like(w)
    hp = qes.HParams(sigma=cfg.sigma, lr=cfg.lr, gamma=cfg.gamma, n_pop=cfg.n_pop)
    seed = int(wl.draw_seeds(1, 1, stream=9)[0, 0])
    tensors = []
    for i, t in enumerate(cfg.tensors):
        d = qes.TensorDesc(bits=4, rows=t.rows, cols=t.cols, group_size=cfg.group_size, elem_offset=t.elem_offset)
        n_sc = t.rows * (t.cols // cfg.group_size)
        sc = torch.from_numpy(np.random.default_rng([wl.MASTER_SEED, 8, i]).lognormal(cfg.scale_mu, cfg.scale_s, n_sc)
                              .astype(np.float16)).cuda()
        x = torch.randn(t.cols, device="cuda", dtype=torch.float16)
        y = torch.empty(t.rows, device="cuda", dtype=torch.float32)
        lo = t.elem_offset // 2
        tensors.append((t, d, w[lo:lo + t.numel // 2], scratch[lo:lo + t.numel // 2], sc, x, y))

    def timed(fn, group):
        """Mean device time of one pass over `group`.  The pass is captured once in a CUDA graph and replayed, so that
        the host's per-call cost (several microseconds through ctypes) does not hide kernels that are shorter than it."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(3):
                for item in group:
                    fn(item)
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for item in group:
                fn(item)
        graph.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.reps):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.reps

    plain = lambda it: qes.qes_gemv(it[1], it[2], it[4], it[5], it[6])
    fused = lambda it: qes.qes_gemv_perturbed(it[1], it[2], it[4], seed, hp, it[5], it[6])
    store = lambda it: qes.qes_perturb(it[1], it[2], it[3], None, seed, hp)
    shapes = {}
    for item in tensors:
        shapes.setdefault(item[0].name.split(".")[-1], []).append(item)
    print(f"{args.workload}: {len(tensors)} tensors, {cfg.numel / 1e9:.3f}e9 codes, HBM peak {hbm:.0f} GB/s ({peak_src})")
    print(f"{'tensors':34s} {'MB read':>9s} {'plain ms':>9s} {'GB/s':>7s} {'of HBM':>7s} {'in-read perturbed ms':>21s} {'ratio':>6s} "
          f"{'qes_perturb (stored copy) ms':>29s}")
    rows = list(shapes.items()) + [("all tensors (one decode step)", tensors)]
    for name, group in rows:
        nbytes = sum(it[0].numel // 2 + it[4].numel() * 2 for it in group)
        t_plain, t_fused, t_store = timed(plain, group), timed(fused, group), timed(store, group)
        gbs = nbytes / t_plain / 1e6
        note = "" if nbytes > L2_BYTES else "  (fits L2)"
        label = f"{name} x{len(group)} {group[0][0].rows}x{group[0][0].cols}" if name in shapes else name
        print(f"{label:34s} {nbytes / 1e6:9.1f} {t_plain:9.3f} {gbs:7.0f} {gbs / hbm:7.2f} {t_fused:21.3f} {t_fused / t_plain:6.1f} "
              f"{t_store:29.3f}{note}")
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
