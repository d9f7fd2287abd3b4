"""CPU-side checks of the C ABI: the library loads, exports what the header declares, and turns
invalid arguments into error codes before anything is launched (no GPU needed for any of it).

The calls that pass made-up device addresses run in a child process that sees no CUDA device
(CUDA_VISIBLE_DEVICES empty): should a validation branch ever regress, the call then ends in
QES_ERR_CUDA instead of a kernel touching an address that was never allocated."""
import ctypes as C
import os
import re
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NO_GPU_ENV = {**os.environ, "CUDA_VISIBLE_DEVICES": ""}


def _run_without_a_device(body: str) -> None:
    code = "import sys; sys.path.insert(0, %r)\n" % ROOT + textwrap.dedent(body)
    r = subprocess.run([sys.executable, "-c", code], env=NO_GPU_ENV, capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr


@pytest.fixture(scope="module")
def lib():
    from paper_2602_03120_b200 import binding, build
    build.build_library()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "qes.h")).read()
    names = re.findall(r"^(?:int|const char\*)\s+(qes_\w+)\s*\(", header, flags=re.M)
    assert set(names) >= {"qes_perturb", "qes_update", "qes_replay_residual", "qes_perturb_pair", "qes_gaussian_factors", "qes_pipe_probe",
                          "qes_gaussian_estimates", "qes_estimate_bounds", "qes_pair_deltas", "qes_gemv", "qes_gemv_perturbed",
                          "qes_replay_fidelity", "qes_pipe_probe_static", "qes_strerror", "qes_version"}
    for n in names:
        assert hasattr(lib, n), n
    assert lib.qes_version() >= 100


def test_struct_layouts_match_header():
    from paper_2602_03120_b200 import binding
    assert C.sizeof(binding._TensorDesc) == 40 and C.sizeof(binding._HParams) == 36
    assert binding._TensorDesc.rows.offset == 16 and binding._TensorDesc.elem_offset.offset == 32


def test_invalid_arguments_are_rejected_without_launching(lib):
    _run_without_a_device("""
    import ctypes as C
    from paper_2602_03120_b200 import binding
    lib = binding.load()

    def call(*, bits=4, rows=4, cols=64, group=0, off=0, qmin=None, qmax=None, sigma=0.5, gamma=0.9, n_pop=4, K=1,
             w=0x1000, seeds=0x2000, fit=0x3000, res=None, unit=0, mode=0, scales=None):
        d = binding.TensorDesc(bits=bits, rows=rows, cols=cols, group_size=group, elem_offset=off, qmin=qmin, qmax=qmax).c()
        h = binding.HParams(sigma=sigma, lr=1.0, gamma=gamma, n_pop=n_pop, sigma_unit=unit, boundary_mode=mode).c()
        return lib.qes_update(C.byref(d), w, scales, seeds, fit, K, res, C.byref(h), None, None)

    assert call(bits=5) == -2
    assert call(cols=48) == -3 and call(rows=0) == -3 and call(group=48) == -3 and call(cols=64, group=128) == -3
    assert call(off=16) == -3
    assert call(w=0x1008) == -4 and call(seeds=0x2004) == -4 and call(res=0x4004, K=0) == -4
    assert call(sigma=0.0) == -5 and call(sigma=-1.0) == -5 and call(n_pop=0) == -5 and call(K=-1) == -5
    assert call(K=(1 << 20) + 1) == -5 and call(K=2**31 - 1) == -5          # replay depth above QES_MAX_K
    assert call(gamma=1.5) == -5 and call(qmin=3, qmax=3) == -5 and call(qmin=-9, qmax=7) == -5
    assert call(unit=2) == -6 and call(mode=7) == -6 and call(res=0x4000, K=2) == -6
    assert call(w=None) == -1 and call(seeds=None) == -1 and call(unit=1, scales=None) == -1
    assert call(n_pop=1067, K=1) == -8 and call(n_pop=1 << 30, K=0) == -8
    d = binding.TensorDesc(bits=4, rows=4, cols=64).c()
    h = binding.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=4).c()
    assert lib.qes_perturb(C.byref(d), None, 0x1000, None, 1, C.byref(h), None) == -1
    assert lib.qes_perturb(None, 0x1000, 0x1000, None, 1, C.byref(h), None) == -1
    assert lib.qes_replay_residual(C.byref(d), 0x1000, None, 0x2000, 0x3000, 2, C.byref(h), None, None) == -1
    assert lib.qes_replay_residual(C.byref(d), 0x1000, None, 0x2000, 0x3000, 2, C.byref(h), 0x4008, None) == -4
    assert lib.qes_replay_residual(C.byref(d), 0x1000, None, 0x2000, 0x3000, (1 << 20) + 1, C.byref(h), 0x4000, None) == -5
    # antithetic pairs: flag must be 0 or 1, the population even, the pair call needs the flag and two outputs
    ha = lambda **kw: binding.HParams(**{**dict(sigma=0.5, lr=1.0, gamma=0.9, n_pop=4, antithetic=1), **kw}).c()
    h2, h3, h1 = ha(antithetic=2), ha(n_pop=3), ha()
    h5 = ha(antithetic=0, noise_mode=2)
    assert lib.qes_update(C.byref(d), 0x1000, None, 0x2000, 0x3000, 1, None, C.byref(h5), None, None) == -6
    h4 = ha(antithetic=0, residual_f16=3)
    assert lib.qes_update(C.byref(d), 0x1000, None, 0x2000, 0x3000, 0, 0x4000, C.byref(h4), None, None) == -6
    assert lib.qes_update(C.byref(d), 0x1000, None, 0x2000, 0x3000, 1, None, C.byref(h2), None, None) == -6
    assert lib.qes_update(C.byref(d), 0x1000, None, 0x2000, 0x3000, 1, None, C.byref(h3), None, None) == -5
    assert lib.qes_perturb_pair(C.byref(d), 0x1000, 0x5000, 0x6000, None, 1, C.byref(h), None) == -6
    assert lib.qes_perturb_pair(C.byref(d), 0x1000, 0x5000, 0x5000, None, 1, C.byref(h1), None) == -6
    assert lib.qes_perturb_pair(C.byref(d), 0x1000, 0x5000, None, None, 1, C.byref(h1), None) == -1
    assert lib.qes_perturb_pair(C.byref(d), 0x1000, 0x5000, 0x6008, None, 1, C.byref(h1), None) == -4
    # the diagnostic entry points validate the same way
    assert lib.qes_gaussian_estimates(0x1000, 0x2000, -1, 0x3000, 0x4000, 0x5000, None) == -3
    assert lib.qes_gaussian_estimates(0x1000, None, 8, 0x3000, 0x4000, 0x5000, None) == -1
    assert lib.qes_gaussian_estimates(0x1002, 0x2000, 8, 0x3000, 0x4000, 0x5000, None) == -4
    assert lib.qes_pair_deltas(0x1000, 0x2000, 0x3000, 0x4000, 8, C.c_float(0.0), 0x5000, 0x6000, None, None) == -5
    assert lib.qes_pair_deltas(0x1000, 0x2000, 0x3000, None, 8, C.c_float(0.5), 0x5000, 0x6000, None, None) == -1
    assert lib.qes_estimate_bounds(None, None, None) == -1
    assert lib.qes_replay_fidelity(C.byref(d), 0x1000, None, None, 0x2000, 0x3000, 0, C.byref(h), 0x7000, None) == -5
    assert lib.qes_replay_fidelity(C.byref(d), 0x1000, None, None, 0x2000, 0x3000, 65, C.byref(h), 0x7000, None) == -5
    assert lib.qes_replay_fidelity(C.byref(d), 0x1000, None, None, 0x2000, 0x3000, 4, C.byref(h), None, None) == -1
    assert lib.qes_replay_fidelity(C.byref(d), 0x1000, 0x5008, None, 0x2000, 0x3000, 4, C.byref(h), 0x7000, None) == -4
    assert lib.qes_gemv(C.byref(d), 0x1000, None, 0x2000, 0x3000, None) == -1
    assert lib.qes_gemv(C.byref(d), 0x1000, 0x4000, 0x2008, 0x3000, None) == -4
    d8 = binding.TensorDesc(bits=8, rows=4, cols=64).c()
    assert lib.qes_gemv(C.byref(d8), 0x1000, 0x4000, 0x2000, 0x3000, None) == -2
    assert lib.qes_gemv_perturbed(C.byref(d), 0x1000, 0x4000, 1, None, 0x2000, 0x3000, None) == -1
    assert lib.qes_gemv_perturbed(C.byref(d), 0x1000, 0x4000, 1, C.byref(h5), 0x2000, 0x3000, None) == -6
    eps, rnd, lim = binding.qes_estimate_bounds()
    assert 0 < eps < 1e-4 and 0 < rnd < 1e-5 and lim > 0xFF000000
    for code in range(-8, 1):
        assert len(lib.qes_strerror(code)) > 1
    # a well-formed call in this process finds no device: an error code, never a launch
    assert call() == -7
    """)


def test_binding_refuses_host_tensors():
    import torch
    from paper_2602_03120_b200 import binding
    d = binding.TensorDesc(bits=4, rows=4, cols=64)
    h = binding.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=4)
    w = torch.zeros(128, dtype=torch.uint8)
    with pytest.raises(binding.QesError):
        binding.qes_perturb(d, w, w, None, 1, h, stream=0)


def test_header_is_plain_c_and_links_from_a_c_program(tmp_path, lib):
    """include/qes.h compiles as C99 on its own, and a C program linked against the library gets the
    documented status codes for invalid arguments (no device needed: validation precedes any CUDA call)."""
    from paper_2602_03120_b200 import binding
    header = os.path.join(ROOT, "include", "qes.h")
    subprocess.run(["gcc", "-x", "c", "-std=c99", "-Wall", "-Wextra", "-Werror", "-fsyntax-only", header], check=True)
    src = tmp_path / "abi.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "qes.h"
int main(void) {
    qes_tensor_desc d; qes_hparams h;
    memset(&d, 0, sizeof d); memset(&h, 0, sizeof h);
    d.bits = 4; d.qmin = -8; d.qmax = 7; d.rows = 4; d.cols = 64;
    h.sigma = 0.5f; h.lr = 1.0f; h.gamma = 0.9f; h.n_pop = 4;
    int a = qes_update(NULL, (void*)0x1000, NULL, (const uint64_t*)0x2000, (const float*)0x3000, 1, NULL, &h, NULL, NULL);
    d.bits = 5;
    int b = qes_update(&d, (void*)0x1000, NULL, (const uint64_t*)0x2000, (const float*)0x3000, 1, NULL, &h, NULL, NULL);
    d.bits = 4; d.cols = 48;
    int c = qes_perturb(&d, (const void*)0x1000, (void*)0x1000, NULL, 1, &h, NULL);
    printf("%d %d %d %d %s\n", qes_version(), a, b, c, qes_strerror(c));
    return 0;
}
''')
    exe = tmp_path / "abi"
    libdir = os.path.dirname(binding.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", f"-I{os.path.join(ROOT, 'include')}", str(src), "-o", str(exe),
                    f"-L{libdir}", "-l:libqes.so", f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True, env=NO_GPU_ENV).stdout.split(maxsplit=4)
    assert int(out[0]) >= 100 and [int(v) for v in out[1:4]] == [-1, -2, -3]
    assert "layout" in out[4]
