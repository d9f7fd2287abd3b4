"""Prints the arithmetic-pipe throughput table of the current GPU (``python -m paper_2602_03120_b200.probe_table``).

Each row is one ``qes_pipe_probe`` kind: best of three runs, in lane-operations (or steps) per second
and in scheduler cycles per warp instruction (or per step) at the GPU's maximum SM clock."""
from __future__ import annotations

import sys

import torch

from . import binding as qes


def main(iters: int = 8192) -> int:
    if not torch.cuda.is_available():
        print("probe_table needs a CUDA device", file=sys.stderr)
        return 1
    qes.load()
    props = torch.cuda.get_device_properties(0)
    mhz = torch.cuda.clock_rate() if hasattr(torch.cuda, "clock_rate") else None
    try:
        import pynvml
        pynvml.nvmlInit()
        mhz = pynvml.nvmlDeviceGetMaxClockInfo(pynvml.nvmlDeviceGetHandleByIndex(0), pynvml.NVML_CLOCK_SM)
    except Exception:
        pass
    mhz = float(mhz or 1965.0)
    lanes = props.multi_processor_count * 128
    print(f"{props.name}: {props.multi_processor_count} SMs, max SM clock {mhz:.0f} MHz, issue peak "
          f"{lanes * mhz * 1e6 / 1e12:.2f} Tlane-op/s")
    print(f"{'kind':>4}  {'instruction(s)':50s} {'T/s':>8}  cycles per warp instruction (or step)")
    for kind, name in qes.PROBE_KINDS.items():
        rate = max(qes.qes_pipe_probe(kind, iters)[0] for _ in range(3))
        print(f"{kind:4d}  {name:50s} {rate / 1e12:8.3f}  {lanes * mhz * 1e6 / rate:6.2f}")
    return 0


if __name__ == "__main__":
    sys.exit(main())
