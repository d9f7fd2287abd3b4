"""qes_pipe_probe on the device at hand: the rates the per-pipe roofline rests on keep their ratios
(fp32 at the issue rate, xor3 and conversions at half, the wide-multiply step at a quarter, the special-function
unit at an eighth), and the operation counts are what the header says."""
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qes():
    import torch
    from paper_2602_03120_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return binding


def _rate(qes, kind, iters=4096):
    return max(qes.qes_pipe_probe(kind, iters)[0] for _ in range(3))


def test_pipe_rates_keep_their_ratios(qes):
    import torch
    props = torch.cuda.get_device_properties(0)
    fma = _rate(qes, 2)
    # one warp instruction per scheduler per cycle is the ceiling: lanes x clock, with the clock below 2.5 GHz
    assert 0.5 * props.multi_processor_count * 128 * 1.0e9 < fma < props.multi_processor_count * 128 * 2.5e9
    for kind, ratio in ((12, 1.0), (13, 1.0), (1, 2.0), (4, 2.0), (7, 2.0), (3, 4.0), (19, 4.0), (9, 8.0), (6, 8.0), (20, 8.0), (21, 8.0), (22, 8.0)):
        r = _rate(qes, kind)
        assert 0.85 * ratio < fma / r < 1.2 * ratio, (kind, fma / r)


def test_operation_counts_and_argument_checks(qes):
    import ctypes as C
    import torch
    props = torch.cuda.get_device_properties(0)
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    ms, ops = C.c_float(0), C.c_double(0)
    lib = qes.load()
    assert lib.qes_pipe_probe(2, 1000, sink.data_ptr(), C.byref(ms), C.byref(ops)) == 0
    assert ops.value == props.multi_processor_count * 8 * 256 * 1000 * 8 and ms.value > 0      # 8 CTAs per SM, 8 chains per thread
    assert lib.qes_pipe_probe(2, 0, sink.data_ptr(), C.byref(ms), C.byref(ops)) == -5
    assert lib.qes_pipe_probe(999, 10, sink.data_ptr(), C.byref(ms), C.byref(ops)) == -6
    assert lib.qes_pipe_probe(2, 10, None, C.byref(ms), C.byref(ops)) == -1
    assert int(sink.item()) == 0                                                              # the sink store is never taken
