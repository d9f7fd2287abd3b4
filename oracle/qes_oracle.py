"""ctypes front end of the CPU oracle (``qes_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may
import this module.  It never touches the CUDA library and shares nothing with it.
Arrays are numpy; packed weights are ``uint8`` (INT4: two codes per byte, even column
in the low nibble; INT8: one two's-complement byte per code), scales are ``float16``
viewed as ``uint16``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qes_oracle.cpp")
_LIB = os.path.join(_HERE, "libqes_oracle.so")

TIER_PLAIN = 0   # double + libm Gaussian
TIER_SPEC = 1    # frozen fp32 operation sequence (what the GPU must reproduce)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ when the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


class _Tensor(C.Structure):
    _fields_ = [("bits", C.c_int32), ("qmin", C.c_int32), ("qmax", C.c_int32), ("group_size", C.c_int32),
                ("rows", C.c_int64), ("cols", C.c_int64), ("elem_offset", C.c_uint64)]


class _HParams(C.Structure):
    _fields_ = [("sigma", C.c_float), ("lr", C.c_float), ("gamma", C.c_float),
                ("n_pop", C.c_int32), ("sigma_unit", C.c_int32), ("boundary_mode", C.c_int32),
                ("antithetic", C.c_int32), ("residual_f16", C.c_int32), ("noise_mode", C.c_int32)]


@dataclass
class Tensor:
    bits: int
    rows: int
    cols: int
    qmin: int | None = None
    qmax: int | None = None
    group_size: int = 0
    elem_offset: int = 0

    def c(self) -> _Tensor:
        qmin = -(1 << (self.bits - 1)) if self.qmin is None else self.qmin
        qmax = (1 << (self.bits - 1)) - 1 if self.qmax is None else self.qmax
        return _Tensor(self.bits, qmin, qmax, self.group_size, self.rows, self.cols, self.elem_offset)

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass
class HParams:
    sigma: float
    lr: float
    gamma: float
    n_pop: int
    sigma_unit: int = 0      # 0 grid steps, 1 weight units (sigma / group scale)
    boundary_mode: int = 0   # 0 gate (Eq. 4), 1 clamp
    antithetic: int = 0      # 1: n_pop / 2 seeded pairs (+delta, -delta); fitness interleaved F+, F-
    residual_f16: int = 0    # 1: the stored residual is binary16
    noise_mode: int = 0      # 0: one Philox call per two elements, 24-bit Bernoulli; 1: per four, 8-bit

    def c(self) -> _HParams:
        return _HParams(self.sigma, self.lr, self.gamma, self.n_pop, self.sigma_unit, self.boundary_mode,
                        self.antithetic, self.residual_f16, self.noise_mode)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.qo_half_to_float.restype = C.c_float
        _lib.qo_half_to_float.argtypes = [C.c_uint16]
        _lib.qo_stochastic_round.restype = C.c_int
        _lib.qo_stochastic_round.argtypes = [C.c_float, C.c_uint32]
        _lib.qo_stochastic_round_byte.restype = C.c_int
        _lib.qo_stochastic_round_byte.argtypes = [C.c_float, C.c_uint32]
        _lib.qo_double_to_half.restype = C.c_uint16
        _lib.qo_double_to_half.argtypes = [C.c_double]
        _lib.qo_applied_step.restype = C.c_longlong
        _lib.qo_applied_step.argtypes = [C.c_int, C.c_longlong, C.c_int, C.c_int, C.c_int]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = _arr(ctr, np.uint32); key = _arr(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().qo_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def bm24(r0, r1):
    """Tier-1 Box-Muller factors: radius, cos, sin (float32) for 32-bit word pairs."""
    r0 = _arr(r0, np.uint32); r1 = _arr(r1, np.uint32)
    n = r0.size
    R = np.empty(n, np.float32); Cs = np.empty(n, np.float32); Sn = np.empty(n, np.float32)
    lib().qo_bm24(_p(r0), _p(r1), C.c_int64(n), _p(R), _p(Cs), _p(Sn))
    return R, Cs, Sn


def stochastic_round(x: float, rword: int) -> int:
    return lib().qo_stochastic_round(C.c_float(x), C.c_uint32(rword))


def stochastic_round_byte(x: float, byte: int) -> int:
    return lib().qo_stochastic_round_byte(C.c_float(x), C.c_uint32(byte))


def half_to_float(h: int) -> float:
    return lib().qo_half_to_float(C.c_uint16(h))


def to_half(values) -> np.ndarray:
    """Rounds doubles to binary16 (nearest even); returns the bit patterns as uint16."""
    v = _arr(values, np.float64).reshape(-1)
    out = np.empty(v.size, np.uint16)
    lib().qo_doubles_to_halves(_p(v), C.c_int64(v.size), _p(out))
    return out


def applied_step(w: int, step: int, qmin: int, qmax: int, mode: int) -> int:
    return lib().qo_applied_step(w, step, qmin, qmax, mode)


def delta(seed: int, J, sigma_eff: float, tier: int = TIER_SPEC, tau: float = 0.0, dmin: int = -8,
          noise_mode: int = 0):
    """Discrete perturbation of global elements J for one seed: (delta int32, x float64, near uint8).
    dmin = -7 gives the symmetric 4-bit range used for antithetic pairs."""
    J = _arr(J, np.uint64)
    n = J.size
    d = np.empty(n, np.int32); x = np.empty(n, np.float64); near = np.empty(n, np.uint8)
    lib().qo_delta(C.c_uint64(seed), _p(J), C.c_int64(n), C.c_float(sigma_eff), C.c_int(tier),
                   C.c_double(tau), C.c_int(dmin), C.c_int(noise_mode), _p(d), _p(x), _p(near))
    return d, x, near


def pair_deltas(r0, r1, r2, r3, sigma_eff: float, dmin: int = -8):
    """delta of the even and odd element of pairs from their four Philox words (default noise mode, tier 1)."""
    r0, r1, r2, r3 = (_arr(r, np.uint32) for r in (r0, r1, r2, r3))
    n = r0.size
    de = np.empty(n, np.int32); do = np.empty(n, np.int32)
    lib().qo_pair_deltas(_p(r0), _p(r1), _p(r2), _p(r3), C.c_int64(n), C.c_float(sigma_eff), C.c_int(dmin), _p(de), _p(do))
    return de, do


def unpack(bits: int, packed, n: int) -> np.ndarray:
    packed = _arr(packed, np.uint8)
    out = np.empty(n, np.int32)
    lib().qo_unpack(C.c_int(bits), _p(packed), C.c_int64(n), _p(out))
    return out


def pack(bits: int, codes) -> np.ndarray:
    codes = _arr(codes, np.int32)
    n = codes.size
    out = np.zeros(n if bits == 8 else n // 2, np.uint8)
    lib().qo_pack(C.c_int(bits), _p(codes), C.c_int64(n), _p(out))
    return out


def _scales(scales):
    if scales is None:
        return None
    s = np.ascontiguousarray(scales)
    if s.dtype == np.float16:
        s = s.view(np.uint16)
    assert s.dtype == np.uint16
    return s


def _idx(idx, t: Tensor):
    if idx is None:
        return None, t.numel
    idx = _arr(idx, np.int64)
    return idx, idx.size


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def perturb(t: Tensor, w, scales, seed: int, hp: HParams, tier=TIER_SPEC, idx=None, nthreads=None, sign: int = 1):
    w = _arr(w, np.uint8); s = _scales(scales); idx, n = _idx(idx, t)
    out = np.empty(n, np.int32)
    tc, hc = t.c(), hp.c()
    rc = lib().qo_perturb(C.byref(tc), _p(w), _p(s), C.c_uint64(seed), C.c_int(sign), C.byref(hc), C.c_int(tier),
                          _p(idx), C.c_int64(n), C.c_int(nthreads or default_threads()), _p(out))
    if rc:
        raise ValueError(f"oracle rejected arguments ({rc})")
    return out


def update(t: Tensor, w, scales, seeds, fitness, K: int, hp: HParams, residual_in=None,
           tier=TIER_SPEC, idx=None, nthreads=None):
    """Algorithm 2 (or Algorithm 1 when residual_in is given and K == 0).

    Returns a dict: w_new int32, e_new float64, band float64 (smallest distance of any
    generation's pre-rounding value to a rounding boundary), gate_final uint8,
    gate_replay int32, attempted uint8, blocked uint64 (bit k: the boundary rule blocked or
    shortened generation k's rounded step) -- one entry per requested element.
    """
    w = _arr(w, np.uint8); s = _scales(scales); idx, n = _idx(idx, t)
    seeds = _arr(seeds, np.uint64).reshape(-1); fitness = _arr(fitness, np.float32).reshape(-1)
    assert fitness.size == (K + 1) * hp.n_pop and seeds.size == fitness.size // (2 if hp.antithetic else 1)
    if residual_in is None:
        res = None
    elif hp.residual_f16:
        res = np.ascontiguousarray(residual_in)
        res = res.view(np.uint16) if res.dtype == np.float16 else res
        assert res.dtype == np.uint16
    else:
        res = _arr(residual_in, np.float32)
    out = dict(w_new=np.empty(n, np.int32), e_new=np.empty(n, np.float64), band=np.empty(n, np.float64),
               gate_final=np.empty(n, np.uint8), gate_replay=np.empty(n, np.int32),
               attempted=np.empty(n, np.uint8), blocked=np.empty(n, np.uint64))
    tc, hc = t.c(), hp.c()
    rc = lib().qo_update(C.byref(tc), _p(w), _p(s), _p(seeds), _p(fitness), C.c_int(K), _p(res),
                         C.byref(hc), C.c_int(tier), _p(idx), C.c_int64(n),
                         C.c_int(nthreads or default_threads()),
                         _p(out["w_new"]), _p(out["e_new"]), _p(out["band"]), _p(out["gate_final"]),
                         _p(out["gate_replay"]), _p(out["attempted"]), _p(out["blocked"]))
    if rc:
        raise ValueError(f"oracle rejected arguments ({rc})")
    return out


def replay_residual(t: Tensor, w, scales, seeds, fitness, K: int, hp: HParams,
                    tier=TIER_SPEC, idx=None, nthreads=None):
    w = _arr(w, np.uint8); s = _scales(scales); idx, n = _idx(idx, t)
    seeds = _arr(seeds, np.uint64).reshape(-1); fitness = _arr(fitness, np.float32).reshape(-1)
    assert fitness.size == K * hp.n_pop and seeds.size == fitness.size // (2 if hp.antithetic else 1)
    out = dict(e=np.empty(n, np.float64), band=np.empty(n, np.float64), gate_replay=np.empty(n, np.int32),
               blocked=np.empty(n, np.uint64))
    tc, hc = t.c(), hp.c()
    rc = lib().qo_replay_residual(C.byref(tc), _p(w), _p(s), _p(seeds), _p(fitness), C.c_int(K),
                                  C.byref(hc), C.c_int(tier), _p(idx), C.c_int64(n),
                                  C.c_int(nthreads or default_threads()),
                                  _p(out["e"]), _p(out["band"]), _p(out["gate_replay"]), _p(out["blocked"]))
    if rc:
        raise ValueError(f"oracle rejected arguments ({rc})")
    return out
