"""qes_pipe_probe_static: the pipe probes for a caller that may not allocate device memory (all of its scratch
is a static device array inside the library).  Its figures must agree with qes_pipe_probe's, which takes its scratch
from the caller -- on two calls in a row, since every call reuses the same array.  Collected last on purpose."""
import ctypes as C

import pytest

pytestmark = pytest.mark.gpu

RATE_TOLERANCE = 0.10      # two timings of the same arithmetic, one by CUDA events, one by the GPU's global timer


@pytest.fixture(scope="module")
def qes():
    import torch
    from paper_2602_03120_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return binding


def test_static_probe_matches_the_probe_with_caller_scratch_twice_in_a_row(qes):
    import torch
    lib = qes.load()
    iters = 4096
    for kind in (2, 1, 19, 9, 8):          # fp32 fma, xor3, wide multiply + xor3, special-function unit, a Philox round
        sink = torch.zeros(1, dtype=torch.int32, device="cuda")
        ms_ref, ops_ref = C.c_float(0), C.c_double(0)
        best_ref = 0.0
        for _ in range(3):
            assert lib.qes_pipe_probe(kind, iters, sink.data_ptr(), C.byref(ms_ref), C.byref(ops_ref)) == 0
            best_ref = max(best_ref, ops_ref.value / ms_ref.value)
        for call in range(2):              # the second call finds the first one's time stamps in the array
            before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
            ms, ops = C.c_float(0), C.c_double(0)
            best = 0.0
            for _ in range(3):
                assert lib.qes_pipe_probe_static(kind, iters, 8, C.byref(ms), C.byref(ops)) == 0
                best = max(best, ops.value / ms.value)
            assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == before
            assert ops.value == ops_ref.value                                   # the same grid, the same work
            assert abs(best / best_ref - 1.0) <= RATE_TOLERANCE, (kind, call, best / best_ref)


def test_static_probe_rejects_what_its_array_cannot_hold(qes):
    import torch
    lib = qes.load()
    ms, ops = C.c_float(-1.0), C.c_double(-1.0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    too_many = 4096 // sms + 1
    assert lib.qes_pipe_probe_static(2, 100, too_many, C.byref(ms), C.byref(ops)) == -8
    assert b"static probe array" in lib.qes_strerror(-8)
    assert lib.qes_pipe_probe_static(2, 100, 0, C.byref(ms), C.byref(ops)) == -5
    assert lib.qes_pipe_probe_static(2, 0, 8, C.byref(ms), C.byref(ops)) == -5
    assert lib.qes_pipe_probe_static(77, 100, 8, C.byref(ms), C.byref(ops)) == -6
    assert lib.qes_pipe_probe_static(2, 100, 8, None, C.byref(ops)) == -1
    assert ms.value == -1.0 and ops.value == -1.0                               # nothing was written on an error
    # the largest grid that fits still runs, and a small one too
    assert lib.qes_pipe_probe_static(2, 256, 4096 // sms, C.byref(ms), C.byref(ops)) == 0 and ms.value > 0
    assert ops.value == sms * (4096 // sms) * 256 * 256 * 8
    assert lib.qes_pipe_probe_static(1, 256, 1, C.byref(ms), C.byref(ops)) == 0 and ms.value > 0
