"""Seeded synthetic inputs for the QES parameter pass.

This module only draws inputs (codes, scales, seeds, rewards) and lists tensor shapes.
It holds none of the method's arithmetic and is the one module that both the CUDA
binding's callers and the CPU oracle's tests may use.  Everything is numpy on the host;
callers move arrays to the device themselves.

The five workloads follow the benchmark configurations: a single 4096x4096 INT4 matrix,
and decoder-shaped weight sets (1.5B / 7B INT4, 7B INT8, 8B INT4) whose linear layers
take the geometry of the models the paper fine-tunes (Sec. 4.1, App. C); the paper's
GPTQ checkpoints and task rewards are replaced by uniform random codes, lognormal
scales and Gaussian / Student-t rewards that are z-scored per generation
(Algorithm 1, the reward-normalisation line of the population loop).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

MASTER_SEED = 0
_STREAM_CODES, _STREAM_SCALES, _STREAM_SEEDS, _STREAM_REWARDS, _STREAM_SAMPLE = 1, 2, 3, 4, 5


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int
    elem_offset: int   # global index of element (0, 0) in the model's flat order

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass(frozen=True)
class Workload:
    name: str
    bits: int
    group_size: int          # 0 = one scale per row
    n_pop: int
    K: int
    sigma: float
    lr: float
    gamma: float
    scale_mu: float
    scale_s: float
    reward_dist: str         # "normal" | "student_t3"
    layers: int
    layer_shapes: tuple      # ((name, rows, cols), ...) per layer
    tensors: tuple = field(default=())

    @property
    def qmin(self) -> int:
        return -(1 << (self.bits - 1))

    @property
    def qmax(self) -> int:
        return (1 << (self.bits - 1)) - 1

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def generations(self) -> int:
        return self.K + 1


def _decoder(hidden: int, kv: int, mlp: int):
    return (("q_proj", hidden, hidden), ("k_proj", kv, hidden), ("v_proj", kv, hidden),
            ("o_proj", hidden, hidden), ("gate_proj", mlp, hidden), ("up_proj", mlp, hidden),
            ("down_proj", hidden, mlp))


def _make(name, bits, group, n_pop, K, layers, shapes, scale_mu=-4.0, scale_s=0.3,
          reward_dist="normal", sigma=0.5, lr=1.0, gamma=0.9) -> Workload:
    tensors, off = [], 0
    for layer in range(layers):
        for (nm, r, c) in shapes:
            tensors.append(TensorSpec(f"layers.{layer}.{nm}" if layers > 1 else nm, r, c, off))
            off += r * c
    return Workload(name, bits, group, n_pop, K, sigma, lr, gamma, scale_mu, scale_s, reward_dist,
                    layers, tuple(shapes), tuple(tensors))


WORKLOADS = {
    "matrix4096_int4": _make("matrix4096_int4", 4, 128, 8, 4, 1, (("weight", 4096, 4096),)),
    "decoder1p5b_int4": _make("decoder1p5b_int4", 4, 128, 16, 8, 28, _decoder(1536, 256, 8960)),
    "decoder7b_int4": _make("decoder7b_int4", 4, 128, 32, 16, 28, _decoder(3584, 512, 18944)),
    "decoder7b_int8": _make("decoder7b_int8", 8, 0, 32, 16, 28, _decoder(3584, 512, 18944), scale_mu=-6.0),
    "decoder8b_int4": _make("decoder8b_int4", 4, 64, 64, 64, 32, _decoder(4096, 1024, 14336),
                            reward_dist="student_t3"),
}
CONFIG_ORDER = ("matrix4096_int4", "decoder1p5b_int4", "decoder7b_int4", "decoder7b_int8", "decoder8b_int4")


def _rng(*stream) -> np.random.Generator:
    return np.random.default_rng([MASTER_SEED, *stream])


def packed_bytes(bits: int, numel: int) -> int:
    return numel if bits == 8 else numel // 2


def draw_codes(wl: Workload, tensor_index: int, numel: int | None = None) -> np.ndarray:
    """Packed uniform random codes (uint8) of one tensor: every byte value equally likely, i.e.
    INT4 codes uniform in [-8, 7] (two per byte) or INT8 codes uniform in [-128, 127]."""
    n = wl.tensors[tensor_index].numel if numel is None else numel
    return _rng(_STREAM_CODES, tensor_index).integers(0, 256, size=packed_bytes(wl.bits, n), dtype=np.uint8)


def draw_scales(wl: Workload, tensor_index: int) -> np.ndarray:
    """fp16 scales, lognormal(mu, s): [rows, cols / group] or [rows] for per-channel grids."""
    t = wl.tensors[tensor_index]
    n = t.rows * (t.cols // wl.group_size) if wl.group_size else t.rows
    return _rng(_STREAM_SCALES, tensor_index).lognormal(wl.scale_mu, wl.scale_s, size=n).astype(np.float16)


def draw_seeds(generations: int, n_pop: int, stream: int = 0) -> np.ndarray:
    """uint64 member seeds [generations, n_pop], oldest generation first."""
    return _rng(_STREAM_SEEDS, stream).integers(0, np.iinfo(np.uint64).max, size=(generations, n_pop),
                                                dtype=np.uint64, endpoint=True)


def draw_fitness(generations: int, n_pop: int, dist: str = "normal", stream: int = 0) -> np.ndarray:
    """Rewards drawn per generation, then z-scored over the population (population std) in
    float64 and cast to float32; an all-equal population maps to zeros."""
    rng = _rng(_STREAM_REWARDS, stream)
    raw = rng.standard_normal((generations, n_pop)) if dist == "normal" else rng.standard_t(3, (generations, n_pop))
    return z_score(raw)


def z_score(raw: np.ndarray) -> np.ndarray:
    raw = np.asarray(raw, np.float64)
    mu = raw.mean(axis=-1, keepdims=True)
    sd = raw.std(axis=-1, keepdims=True)
    out = np.where(sd > 0, (raw - mu) / np.where(sd > 0, sd, 1.0), 0.0)
    return out.astype(np.float32)


def sample_elements(numel: int, count: int, stream: int = 0, word: int = 32) -> np.ndarray:
    """Sorted element indices for sampled parity: the first and last `word` elements of the tensor
    plus whole `word`-element groups drawn uniformly."""
    rng = _rng(_STREAM_SAMPLE, stream)
    n_words = numel // word
    picks = rng.integers(0, n_words, size=max(0, count // word - 2))
    words = np.unique(np.concatenate([[0, n_words - 1], picks]))
    return (words[:, None] * word + np.arange(word)[None, :]).reshape(-1).astype(np.int64)
