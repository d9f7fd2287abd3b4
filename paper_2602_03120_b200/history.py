"""The optimizer state of Stateless Seed Replay (Sec. 3.3, Algorithm 2): a window of the last K
generations' seeds and normalised rewards, H_t = {(S_tau, F_tau)} for tau = t-K .. t-1.

Host-side bookkeeping only (no arithmetic of the method): it keeps the window, lays it out as the
generation-major, oldest-first tables the library expects, and serialises to a few kilobytes --
12 bytes per (generation, member) with one seed per member, so K = 50, N = 50 is 30,000 bytes,
the "≈29.7 KB" of the paper's memory table."""
from __future__ import annotations

import numpy as np


class SeedHistory:
    def __init__(self, window: int, n_pop: int, seeds_per_generation: int | None = None):
        if window < 0 or n_pop <= 0:
            raise ValueError("window must be >= 0 and n_pop > 0")
        self.window, self.n_pop = int(window), int(n_pop)
        self.n_seeds = int(seeds_per_generation if seeds_per_generation is not None else n_pop)
        self._seeds: list[np.ndarray] = []      # oldest first
        self._fitness: list[np.ndarray] = []

    def __len__(self) -> int:
        return len(self._seeds)

    def tables(self, seeds_now, fitness_now):
        """(seeds [(k+1) * n_seeds] uint64, fitness [(k+1) * n_pop] float32, k): the window's k <= K
        generations oldest first, then the current generation -- the arguments of ``qes_update``."""
        s_now, f_now = self._check(seeds_now, fitness_now)
        seeds = np.concatenate(self._seeds + [s_now]) if self._seeds else s_now.copy()
        fitness = np.concatenate(self._fitness + [f_now]) if self._fitness else f_now.copy()
        return seeds, fitness, len(self._seeds)

    def push(self, seeds_now, fitness_now) -> None:
        """Algorithm 2, last line (the current seeds and rewards join the history): the oldest generation leaves once the window is full."""
        s_now, f_now = self._check(seeds_now, fitness_now)
        if self.window == 0:
            return
        self._seeds.append(s_now.copy()); self._fitness.append(f_now.copy())
        if len(self._seeds) > self.window:
            self._seeds.pop(0); self._fitness.pop(0)

    def _check(self, seeds_now, fitness_now):
        s = np.ascontiguousarray(seeds_now, dtype=np.uint64).reshape(-1)
        f = np.ascontiguousarray(fitness_now, dtype=np.float32).reshape(-1)
        if s.size != self.n_seeds or f.size != self.n_pop:
            raise ValueError(f"expected {self.n_seeds} seeds and {self.n_pop} fitness values, got {s.size} and {f.size}")
        return s, f

    @property
    def nbytes(self) -> int:
        return sum(a.nbytes for a in self._seeds) + sum(a.nbytes for a in self._fitness)

    def to_bytes(self) -> bytes:
        head = np.array([self.window, self.n_pop, self.n_seeds, len(self._seeds)], dtype=np.int64).tobytes()
        return head + b"".join(a.tobytes() for a in self._seeds) + b"".join(a.tobytes() for a in self._fitness)

    @classmethod
    def from_bytes(cls, blob: bytes) -> "SeedHistory":
        window, n_pop, n_seeds, k = (int(v) for v in np.frombuffer(blob[:32], dtype=np.int64))
        h = cls(window, n_pop, n_seeds)
        off = 32
        for _ in range(k):
            h._seeds.append(np.frombuffer(blob[off:off + 8 * n_seeds], dtype=np.uint64).copy()); off += 8 * n_seeds
        for _ in range(k):
            h._fitness.append(np.frombuffer(blob[off:off + 4 * n_pop], dtype=np.float32).copy()); off += 4 * n_pop
        if off != len(blob):
            raise ValueError("trailing bytes in a serialised history")
        return h
