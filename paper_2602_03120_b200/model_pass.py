"""A whole weight set on one GPU: flat packed buffer, per-tensor descriptors, and the three passes.

This is the call a user of the library makes for a model: ``perturb_member`` (Algorithm 1, member
loop), ``update`` (Algorithm 2) and ``replay_residual`` launch one library call per tensor -- or, when
sigma is in grid units and the kernels need no per-tensor geometry, per run of consecutive tensors
-- on the current stream.  Nothing here computes: every step runs in the kernels behind the C ABI.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as qes
from . import workloads as wl


def shard_tensors(workload: wl.Workload, rank: int, world: int):
    """Weak-scaling shard: rank r owns copy r of the decoder stack of a `world`-times deeper model.
    Global element offsets continue across ranks, so every rank draws a disjoint noise stream and the
    union equals one model of world*layers layers updated on one device.  No data is exchanged."""
    per_rank = workload.numel
    return tuple(wl.TensorSpec(f"shard{rank}.{t.name}", t.rows, t.cols, t.elem_offset + rank * per_rank)
                 for t in workload.tensors)


MAX_SEGMENT_ELEMS = 1 << 28   # one launch covers at most this many codes (a few hundred ms of work)


def launch_segments(tensors, max_elems: int = MAX_SEGMENT_ELEMS):
    """Groups consecutive tensors into launches of at most `max_elems` codes.  With sigma in grid
    units the kernels never look at rows, columns or scales: noise depends only on the global
    element index, so any contiguous run of tensors can be passed as one [numel / 32, 32] tensor.
    Returns (first_tensor_index, elem_offset, numel) triples; a tensor larger than the limit is a
    segment of its own."""
    segs, start, off, n = [], 0, None, 0
    for i, t in enumerate(tensors):
        if n and (n + t.numel > max_elems or t.elem_offset != off + n):
            segs.append((start, off, n)); n = 0
        if n == 0:
            start, off = i, t.elem_offset
        n += t.numel
    if n:
        segs.append((start, off, n))
    return segs


class ModelPass:
    def __init__(self, workload: wl.Workload, device="cuda", rank: int = 0, world: int = 1,
                 sigma_unit: int = qes.SIGMA_GRID, with_scales: bool = False, tensors=None,
                 antithetic: bool = False, noise_mode: int = qes.NOISE_PAIR24):
        self.wl = workload
        self.device = torch.device(device)
        self.tensors = tuple(tensors) if tensors is not None else shard_tensors(workload, rank, world)
        self.base = self.tensors[0].elem_offset
        self.numel = sum(t.numel for t in self.tensors)
        self.bytes = wl.packed_bytes(workload.bits, self.numel)
        self.w = torch.empty(self.bytes, dtype=torch.uint8, device=self.device)
        self.hp = qes.HParams(sigma=workload.sigma, lr=workload.lr, gamma=workload.gamma, n_pop=workload.n_pop,
                              sigma_unit=sigma_unit, antithetic=int(antithetic), noise_mode=noise_mode)
        self.descs = [qes.TensorDesc(bits=workload.bits, rows=t.rows, cols=t.cols, group_size=workload.group_size,
                                     elem_offset=t.elem_offset) for t in self.tensors]
        # grid-unit sigma: fused launches over runs of tensors; weight-unit sigma: one launch per tensor
        self.fused = sigma_unit == qes.SIGMA_GRID
        self.segments = [(wl.TensorSpec(f"segment{j}", n // 32, 32, off),
                          qes.TensorDesc(bits=workload.bits, rows=n // 32, cols=32, group_size=0, elem_offset=off))
                         for j, (_, off, n) in enumerate(launch_segments(self.tensors))]
        self.scales = None
        if with_scales or sigma_unit == qes.SIGMA_WEIGHT:
            self.scales = [torch.from_numpy(wl.draw_scales(workload, i)).to(self.device)
                           for i in range(len(self.tensors))]

    def _slice(self, buf, t):
        lo = wl.packed_bytes(self.wl.bits, t.elem_offset - self.base)
        return buf[lo:lo + wl.packed_bytes(self.wl.bits, t.numel)]

    def host_codes(self) -> np.ndarray:
        """Packed synthetic codes of this shard on the host (uniform random bytes per tensor)."""
        out = np.empty(self.bytes, np.uint8)
        for i, t in enumerate(self.tensors):
            lo = wl.packed_bytes(self.wl.bits, t.elem_offset - self.base)
            out[lo:lo + wl.packed_bytes(self.wl.bits, t.numel)] = wl.draw_codes(self.wl, i)
        return out

    def load(self, host_packed) -> None:
        self.w.copy_(host_packed if isinstance(host_packed, torch.Tensor) else torch.from_numpy(host_packed),
                     non_blocking=True)

    def _sc(self, i):
        return None if self.scales is None else self.scales[i]

    def _launches(self):
        """(tensor spec, descriptor, scales) per library call."""
        if self.fused:
            return [(t, d, None) for t, d in self.segments]
        return [(t, d, self._sc(i)) for i, (t, d) in enumerate(zip(self.tensors, self.descs))]

    def perturb_member(self, out: torch.Tensor, seed: int) -> int:
        calls = self._launches()
        for t, d, sc in calls:
            qes.qes_perturb(d, self._slice(self.w, t), self._slice(out, t), sc, seed, self.hp)
        return len(calls)

    def perturb_pair(self, out_plus: torch.Tensor, out_minus: torch.Tensor, seed: int) -> int:
        """Both members of one antithetic pair (App. A) from one noise pass."""
        calls = self._launches()
        for t, d, sc in calls:
            qes.qes_perturb_pair(d, self._slice(self.w, t), self._slice(out_plus, t), self._slice(out_minus, t), sc,
                                 seed, self.hp)
        return len(calls)

    def update(self, seeds: torch.Tensor, fitness: torch.Tensor, K: int, stats=None) -> int:
        calls = self._launches()
        for t, d, sc in calls:
            qes.qes_update(d, self._slice(self.w, t), sc, seeds, fitness, K, None, self.hp, stats=stats)
        return len(calls)

    def replay_residual(self, seeds: torch.Tensor, fitness: torch.Tensor, K: int, out: torch.Tensor) -> int:
        calls = self._launches()
        for t, d, sc in calls:
            lo = t.elem_offset - self.base
            qes.qes_replay_residual(d, self._slice(self.w, t), sc, seeds, fitness, K, self.hp, out[lo:lo + t.numel])
        return len(calls)

    def step_from_host(self, host_in: torch.Tensor, host_out: torch.Tensor, scratch: torch.Tensor, member_seeds,
                       seeds: torch.Tensor, fitness: torch.Tensor, K: int, scratch_minus: torch.Tensor | None = None) -> int:
        """One full step (the perturbation of every member, then the stateless update) with the weights
        starting and ending in pinned host memory.  The set is walked launch by launch: the copy-in of
        the next run of tensors and the copy-out of the previous one ride on two side streams under the
        arithmetic of the current one, so only the first copy-in and the last copy-out are exposed."""
        main = torch.cuda.current_stream()
        if not hasattr(self, "_copy_in"):
            self._copy_in, self._copy_out = torch.cuda.Stream(), torch.cuda.Stream()
        calls = self._launches()
        self._copy_in.wait_stream(main)          # the previous step's kernels are done with self.w
        self._copy_out.wait_stream(main)
        arrived = []
        for t, _, _ in calls:
            with torch.cuda.stream(self._copy_in):
                self._slice(self.w, t).copy_(self._slice(host_in, t), non_blocking=True)
                ev = torch.cuda.Event(); ev.record(self._copy_in); arrived.append(ev)
        n = 0
        for (t, d, sc), ev in zip(calls, arrived):
            main.wait_event(ev)
            w_t = self._slice(self.w, t)
            for s in member_seeds:                                   # Algorithm 1, member loop
                if scratch_minus is not None:
                    qes.qes_perturb_pair(d, w_t, self._slice(scratch, t), self._slice(scratch_minus, t), sc, s, self.hp)
                else:
                    qes.qes_perturb(d, w_t, self._slice(scratch, t), sc, s, self.hp)
            qes.qes_update(d, w_t, sc, seeds, fitness, K, None, self.hp)     # Algorithm 2
            n += len(member_seeds) + 1
            done = torch.cuda.Event(); done.record(main)
            with torch.cuda.stream(self._copy_out):
                self._copy_out.wait_event(done)
                self._slice(host_out, t).copy_(w_t, non_blocking=True)
        main.wait_stream(self._copy_out)         # the step ends when the last bytes are back on the host
        return n
