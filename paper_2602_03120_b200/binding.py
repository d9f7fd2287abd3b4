"""Thin ctypes binding of ``libqes.so``: argument marshalling only.

Every step of the parameter pass runs inside the CUDA kernels of the library; this module turns
torch CUDA tensors into device pointers, fills the two C structs and raises on error codes.  It
never falls back to another implementation: a missing library is an ImportError-like failure.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqes.so")

SIGMA_GRID, SIGMA_WEIGHT = 0, 1
BOUNDARY_GATE, BOUNDARY_CLAMP = 0, 1
NOISE_PAIR24, NOISE_QUAD8 = 0, 1


class QesError(RuntimeError):
    pass


class _TensorDesc(C.Structure):
    _fields_ = [("bits", C.c_int32), ("qmin", C.c_int32), ("qmax", C.c_int32), ("group_size", C.c_int32),
                ("rows", C.c_int64), ("cols", C.c_int64), ("elem_offset", C.c_uint64)]


class _HParams(C.Structure):
    _fields_ = [("sigma", C.c_float), ("lr", C.c_float), ("gamma", C.c_float),
                ("n_pop", C.c_int32), ("sigma_unit", C.c_int32), ("boundary_mode", C.c_int32),
                ("antithetic", C.c_int32), ("residual_f16", C.c_int32), ("noise_mode", C.c_int32)]


@dataclass
class TensorDesc:
    bits: int
    rows: int
    cols: int
    qmin: int | None = None
    qmax: int | None = None
    group_size: int = 0
    elem_offset: int = 0

    def c(self) -> _TensorDesc:
        qmin = -(1 << (self.bits - 1)) if self.qmin is None else self.qmin
        qmax = (1 << (self.bits - 1)) - 1 if self.qmax is None else self.qmax
        return _TensorDesc(self.bits, qmin, qmax, self.group_size, self.rows, self.cols, self.elem_offset)

    @property
    def numel(self) -> int:
        return self.rows * self.cols

    @property
    def packed_bytes(self) -> int:
        return self.numel if self.bits == 8 else self.numel // 2


@dataclass
class HParams:
    sigma: float
    lr: float
    gamma: float
    n_pop: int
    sigma_unit: int = SIGMA_GRID
    boundary_mode: int = BOUNDARY_GATE
    antithetic: int = 0
    residual_f16: int = 0
    noise_mode: int = NOISE_PAIR24

    def c(self) -> _HParams:
        return _HParams(self.sigma, self.lr, self.gamma, self.n_pop, self.sigma_unit, self.boundary_mode,
                        self.antithetic, self.residual_f16, self.noise_mode)

    @property
    def residual_dtype(self):
        return torch.float16 if self.residual_f16 else torch.float32

    @property
    def residual_itemsize(self) -> int:
        return 2 if self.residual_f16 else 4

    @property
    def seeds_per_generation(self) -> int:
        return self.n_pop // 2 if self.antithetic else self.n_pop


_lib = None


def load() -> C.CDLL:
    """Load the compiled library; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise QesError(f"{LIB_PATH} is missing: run paper_2602_03120_b200.build.build_library() "
                           "(nvcc, sm_100a); the parameter pass has no fallback implementation")
        lib = C.CDLL(LIB_PATH)
        vp, u64, i32 = C.c_void_p, C.c_uint64, C.c_int32
        lib.qes_perturb.restype = C.c_int
        lib.qes_perturb.argtypes = [C.POINTER(_TensorDesc), vp, vp, vp, u64, C.POINTER(_HParams), vp]
        lib.qes_perturb_pair.restype = C.c_int
        lib.qes_perturb_pair.argtypes = [C.POINTER(_TensorDesc), vp, vp, vp, vp, u64, C.POINTER(_HParams), vp]
        lib.qes_replay_residual.restype = C.c_int
        lib.qes_replay_residual.argtypes = [C.POINTER(_TensorDesc), vp, vp, vp, vp, i32, C.POINTER(_HParams), vp, vp]
        lib.qes_update.restype = C.c_int
        lib.qes_update.argtypes = [C.POINTER(_TensorDesc), vp, vp, vp, vp, i32, vp, C.POINTER(_HParams), vp, vp]
        lib.qes_gaussian_factors.restype = C.c_int
        lib.qes_gaussian_factors.argtypes = [vp, vp, C.c_int64, vp, vp, vp, vp]
        lib.qes_gaussian_estimates.restype = C.c_int
        lib.qes_gaussian_estimates.argtypes = [vp, vp, C.c_int64, vp, vp, vp, vp]
        lib.qes_estimate_bounds.restype = C.c_int
        lib.qes_estimate_bounds.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_uint32)]
        lib.qes_pair_deltas.restype = C.c_int
        lib.qes_pair_deltas.argtypes = [vp, vp, vp, vp, C.c_int64, C.c_float, vp, vp, vp, vp]
        lib.qes_replay_fidelity.restype = C.c_int
        lib.qes_replay_fidelity.argtypes = [C.POINTER(_TensorDesc), vp, vp, vp, vp, vp, i32, C.POINTER(_HParams), vp, vp]
        lib.qes_gemv.restype = C.c_int
        lib.qes_gemv.argtypes = [C.POINTER(_TensorDesc), vp, vp, vp, vp, vp]
        lib.qes_gemv_perturbed.restype = C.c_int
        lib.qes_gemv_perturbed.argtypes = [C.POINTER(_TensorDesc), vp, vp, u64, C.POINTER(_HParams), vp, vp, vp]
        lib.qes_pipe_probe.restype = C.c_int
        lib.qes_pipe_probe.argtypes = [i32, i32, vp, C.POINTER(C.c_float), C.POINTER(C.c_double)]
        lib.qes_pipe_probe_static.restype = C.c_int
        lib.qes_pipe_probe_static.argtypes = [i32, i32, i32, C.POINTER(C.c_float), C.POINTER(C.c_double)]
        lib.qes_strerror.restype = C.c_char_p
        lib.qes_strerror.argtypes = [C.c_int]
        lib.qes_version.restype = C.c_int
        _lib = lib
    return _lib


def _ptr(t, *, dtype=None, nbytes=None, name="tensor"):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise QesError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise QesError(f"{name} must be contiguous")
    if dtype is not None and t.dtype not in (dtype if isinstance(dtype, tuple) else (dtype,)):
        raise QesError(f"{name} has dtype {t.dtype}, expected {dtype}")
    if nbytes is not None and t.numel() * t.element_size() < nbytes:
        raise QesError(f"{name} holds {t.numel() * t.element_size()} bytes, needs {nbytes}")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc: int):
    if rc != 0:
        raise QesError(f"libqes error {rc}: {load().qes_strerror(rc).decode()}")


_W = (torch.uint8, torch.int8)
_S = (torch.float16,)
_SEEDS = (torch.int64, torch.uint64)


def _scale_bytes(d: TensorDesc) -> int:
    return 2 * (d.rows * (d.cols // d.group_size) if d.group_size else d.rows)


def qes_perturb(desc: TensorDesc, w_in, w_out, scales_f16, seed: int, hparams: HParams, stream=None) -> None:
    """W' = Gate(W + delta_i) for one member (Algorithm 1; Eqs. 3-4).  Enqueues, does not synchronise."""
    d, h = desc.c(), hparams.c()
    rc = load().qes_perturb(C.byref(d), _ptr(w_in, dtype=_W, nbytes=desc.packed_bytes, name="w_in"),
                            _ptr(w_out, dtype=_W, nbytes=desc.packed_bytes, name="w_out"),
                            _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                            C.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), C.byref(h), _stream(stream))
    _check(rc)


def qes_perturb_pair(desc: TensorDesc, w_in, w_plus_out, w_minus_out, scales_f16, seed: int, hparams: HParams,
                     stream=None) -> None:
    """Both members of one antithetic pair (App. A): Gate(W + delta) and Gate(W - delta) from one noise pass."""
    d, h = desc.c(), hparams.c()
    rc = load().qes_perturb_pair(C.byref(d), _ptr(w_in, dtype=_W, nbytes=desc.packed_bytes, name="w_in"),
                                 _ptr(w_plus_out, dtype=_W, nbytes=desc.packed_bytes, name="w_plus_out"),
                                 _ptr(w_minus_out, dtype=_W, nbytes=desc.packed_bytes, name="w_minus_out"),
                                 _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                                 C.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), C.byref(h), _stream(stream))
    _check(rc)


def qes_replay_residual(desc: TensorDesc, w, scales_f16, seeds, fitness, K: int, hparams: HParams,
                        residual_out, stream=None) -> None:
    """History loop of Algorithm 2: writes the proxy residual after K generations (fp32)."""
    d, h = desc.c(), hparams.c()
    n, ns = K * hparams.n_pop, K * hparams.seeds_per_generation
    rc = load().qes_replay_residual(C.byref(d), _ptr(w, dtype=_W, nbytes=desc.packed_bytes, name="w"),
                                    _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                                    _ptr(seeds, dtype=_SEEDS, nbytes=8 * ns, name="seeds"),
                                    _ptr(fitness, dtype=torch.float32, nbytes=4 * n, name="fitness"),
                                    K, C.byref(h),
                                    _ptr(residual_out, dtype=hparams.residual_dtype, nbytes=hparams.residual_itemsize * desc.numel,
                                         name="residual_out"),
                                    _stream(stream))
    _check(rc)


def qes_update(desc: TensorDesc, w_inout, scales_f16, seeds, fitness, K: int, residual_inout,
               hparams: HParams, stats=None, stream=None) -> None:
    """In-place update: stateless with seed replay (Algorithm 2) or with a stored residual (Algorithm 1)."""
    d, h = desc.c(), hparams.c()
    n, ns = (K + 1) * hparams.n_pop, (K + 1) * hparams.seeds_per_generation
    rc = load().qes_update(C.byref(d), _ptr(w_inout, dtype=_W, nbytes=desc.packed_bytes, name="w_inout"),
                           _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                           _ptr(seeds, dtype=_SEEDS, nbytes=8 * ns, name="seeds"),
                           _ptr(fitness, dtype=torch.float32, nbytes=4 * n, name="fitness"),
                           K, _ptr(residual_inout, dtype=hparams.residual_dtype,
                                   nbytes=hparams.residual_itemsize * desc.numel, name="residual_inout"),
                           C.byref(h), _ptr(stats, dtype=_SEEDS, nbytes=32, name="stats"), _stream(stream))
    _check(rc)


def qes_gaussian_factors(r0, r1, radius, cosine, sine, stream=None) -> None:
    """Box-Muller factors of the noise contract for 32-bit word pairs (uint32/int32 in, float32 out)."""
    n = r0.numel()
    words = (torch.int32, torch.uint32)
    rc = load().qes_gaussian_factors(_ptr(r0, dtype=words, nbytes=4 * n, name="r0"), _ptr(r1, dtype=words, nbytes=4 * n, name="r1"),
                                     n, _ptr(radius, dtype=torch.float32, nbytes=4 * n, name="radius"),
                                     _ptr(cosine, dtype=torch.float32, nbytes=4 * n, name="cosine"),
                                     _ptr(sine, dtype=torch.float32, nbytes=4 * n, name="sine"), _stream(stream))
    _check(rc)


def qes_replay_fidelity(desc: TensorDesc, w_start, w_end_out, scales_f16, seeds, fitness, generations: int,
                        hparams: HParams, counts, stream=None) -> None:
    """Gate-mismatch count of Stateless Seed Replay against a stored-residual run over `generations` steps (Sec. 3.3)."""
    d, h = desc.c(), hparams.c()
    n, ns = generations * hparams.n_pop, generations * hparams.seeds_per_generation
    rc = load().qes_replay_fidelity(C.byref(d), _ptr(w_start, dtype=_W, nbytes=desc.packed_bytes, name="w_start"),
                                    _ptr(w_end_out, dtype=_W, nbytes=desc.packed_bytes, name="w_end_out"),
                                    _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                                    _ptr(seeds, dtype=_SEEDS, nbytes=8 * ns, name="seeds"),
                                    _ptr(fitness, dtype=torch.float32, nbytes=4 * n, name="fitness"), generations, C.byref(h),
                                    _ptr(counts, dtype=_SEEDS, nbytes=32, name="counts"), _stream(stream))
    _check(rc)


def qes_gemv(desc: TensorDesc, w, scales_f16, x_f16, y, stream=None) -> None:
    """y = (scales * W) x for one packed INT4 tensor (batch 1, fp16 activations, fp32 result)."""
    d = desc.c()
    rc = load().qes_gemv(C.byref(d), _ptr(w, dtype=_W, nbytes=desc.packed_bytes, name="w"),
                         _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                         _ptr(x_f16, dtype=torch.float16, nbytes=2 * desc.cols, name="x"),
                         _ptr(y, dtype=torch.float32, nbytes=4 * desc.rows, name="y"), _stream(stream))
    _check(rc)


def qes_gemv_perturbed(desc: TensorDesc, w, scales_f16, seed: int, hparams: HParams, x_f16, y, stream=None) -> None:
    """The same product over Gate(W + delta(seed)) with the perturbation generated inside the weight read."""
    d, h = desc.c(), hparams.c()
    rc = load().qes_gemv_perturbed(C.byref(d), _ptr(w, dtype=_W, nbytes=desc.packed_bytes, name="w"),
                                   _ptr(scales_f16, dtype=_S, nbytes=_scale_bytes(desc), name="scales"),
                                   C.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), C.byref(h),
                                   _ptr(x_f16, dtype=torch.float16, nbytes=2 * desc.cols, name="x"),
                                   _ptr(y, dtype=torch.float32, nbytes=4 * desc.rows, name="y"), _stream(stream))
    _check(rc)


def qes_gaussian_estimates(r0, r1, radius, cosine, sine, stream=None) -> None:
    """The special-function-unit estimates of the same three factors (what the kernels try first)."""
    n = r0.numel()
    words = (torch.int32, torch.uint32)
    rc = load().qes_gaussian_estimates(_ptr(r0, dtype=words, nbytes=4 * n, name="r0"), _ptr(r1, dtype=words, nbytes=4 * n, name="r1"),
                                       n, _ptr(radius, dtype=torch.float32, nbytes=4 * n, name="radius"),
                                       _ptr(cosine, dtype=torch.float32, nbytes=4 * n, name="cosine"),
                                       _ptr(sine, dtype=torch.float32, nbytes=4 * n, name="sine"), _stream(stream))
    _check(rc)


def qes_estimate_bounds():
    """(eps_bound, rounding_bound, radius_word_limit) of the estimate-then-verify sequence."""
    eps, rnd, lim = C.c_float(0), C.c_float(0), C.c_uint32(0)
    _check(load().qes_estimate_bounds(C.byref(eps), C.byref(rnd), C.byref(lim)))
    return eps.value, rnd.value, lim.value


def qes_pair_deltas(r0, r1, r2, r3, sigma_eff: float, delta_even, delta_odd, verified=None, stream=None) -> None:
    """Eq. 3 for both elements of pairs given their four Philox words, through the kernels' own sequence."""
    n = r0.numel()
    words = (torch.int32, torch.uint32)
    rc = load().qes_pair_deltas(*(_ptr(r, dtype=words, nbytes=4 * n, name=f"r{i}") for i, r in enumerate((r0, r1, r2, r3))),
                                n, C.c_float(sigma_eff), _ptr(delta_even, dtype=torch.int8, nbytes=n, name="delta_even"),
                                _ptr(delta_odd, dtype=torch.int8, nbytes=n, name="delta_odd"),
                                _ptr(verified, dtype=torch.uint8, nbytes=n, name="verified"), _stream(stream))
    _check(rc)


PROBE_KINDS = {0: "mul.wide.u32", 1: "lop3.xor3", 2: "fma.rn.f32", 3: "mul.hi.u32", 4: "cvt.rn.f32.u32",
               5: "sqrt.rn.f32", 6: "cvt.rmi.f32.f32", 7: "mad.lo.u32", 8: "philox round (2 mul.wide + 2 xor3)",
               9: "rsqrt.approx.f32", 10: "add.u32", 11: "shr.u32", 12: "add.rn.f32", 13: "mul.rn.f32",
               14: "setp.lt.f32 + selp", 15: "min.f32", 16: "cvt.rzi.s32.f32", 17: "set.lt.f32 (1.0/0.0)", 18: "mad.wide.u32 (64-bit result live)",
               19: "mul.wide.u32 + xor3 of both halves (steps)", 20: "lg2.approx.f32", 21: "sin.approx.f32",
               22: "sqrt.approx.f32", 23: "cvt.rn.f32.s8"}


def qes_pipe_probe(kind: int, iters: int = 4096):
    """Lane-operations per second of one instruction kind on the current device (synchronises)."""
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    ms, ops = C.c_float(0), C.c_double(0)
    torch.cuda.synchronize()
    _check(load().qes_pipe_probe(kind, iters, sink.data_ptr(), C.byref(ms), C.byref(ops)))
    return ops.value / (ms.value * 1e-3), ms.value


def qes_pipe_probe_static(kind: int, iters: int = 4096, ctas_per_sm: int = 8):
    """qes_pipe_probe without any allocation: scratch and timing live in a static device array inside the library
    (for callers whose device memory belongs to another allocator).  Returns (lane-operations per second, ms)."""
    ms, ops = C.c_float(0), C.c_double(0)
    _check(load().qes_pipe_probe_static(kind, iters, ctas_per_sm, C.byref(ms), C.byref(ops)))
    return ops.value / (ms.value * 1e-3), ms.value
