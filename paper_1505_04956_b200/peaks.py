"""Issue-rate probes behind the notes on the kernels (python -m paper_1505_04956_b200.peaks).

Prints, for the instruction kinds the worker kernels are made of, the cycles one of an SM's four schedulers
spends per warp instruction on this GPU: alone and in the mixes the streaming kernel issues.  The numbers are
what the cost estimates of the kernels are computed from (for instance: a packed two-wide FMA costs as much as
two scalar ones; a min/max, a logic op, a compare or an integer multiply-add runs at half rate; a legacy
tensor-core product holds the tensor pipe for eight cycles and the scheduler for about four).
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

NAMES = ("FFMA (two immediates)", "FFMA acc = x * w + acc", "FFMA2 acc = x * w + acc (two-wide)", "FADD2 (two-wide)",
         "LOP3", "FMNMX", "FSET", "IMAD", "mma.sync m16n8k8 TF32", "LOP3 + FFMA alternating", "LOP3 + FFMA2 alternating",
         "1 mma.sync + 6 FFMA", "1 mma.sync + 4 LOP3")


def issue_rates():
    """Cycles per warp instruction and scheduler, in the order of NAMES (needs a B200)."""
    import torch
    lib = C.CDLL(_build.build_probe())
    lib.asgd_probe_issue_rates.argtypes = [C.POINTER(C.c_float), C.c_int, C.c_void_p, C.c_int]
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    scratch = torch.empty(1 + sms * 512, dtype=torch.float32, device="cuda")
    out = (C.c_float * len(NAMES))()
    rc = lib.asgd_probe_issue_rates(out, len(NAMES), C.c_void_p(scratch.data_ptr()), sms)
    if rc != 0:
        raise RuntimeError("asgd_probe_issue_rates failed (%d)" % rc)
    return [float(v) for v in out]


MMA_NAMES = ("tcgen05.mma 128x256x16 f16, one pair of chunks", "tcgen05.mma 128x256x16, walking four chunks",
             "tcgen05.mma 128x256x16, walking, commit every 4", "tcgen05.mma 128x128x16 f16, one pair of chunks",
             "tcgen05.mma 128x128x16, walking four chunks", "tcgen05.mma 128x128x16, walking, commit every 4",
             "N=256 commit every 4, eight barriers in turn", "N=256 commit every 4, fresh accumulator after a commit",
             "N=256 commit every 16", "N=256 commit every 16, eight barriers in turn", "N=256 two issuing threads, commit every 4",
             "N=256 two issuing threads, no commits")


def mma_rates():
    """Cycles per tcgen05.mma issued back to back by one thread, in the order of MMA_NAMES (needs a B200)."""
    import torch
    lib = C.CDLL(_build.build_probe())
    lib.asgd_probe_mma_rates.argtypes = [C.POINTER(C.c_float), C.c_int, C.c_void_p, C.c_int]
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    scratch = torch.empty(sms, dtype=torch.float32, device="cuda")
    out = (C.c_float * len(MMA_NAMES))()
    rc = lib.asgd_probe_mma_rates(out, len(MMA_NAMES), C.c_void_p(scratch.data_ptr()), sms)
    if rc != 0:
        raise RuntimeError("asgd_probe_mma_rates failed (%d)" % rc)
    return [float(v) for v in out]


if __name__ == "__main__":
    for name, v in zip(NAMES, issue_rates()):
        print("%-48s %7.2f cycles per warp instruction and scheduler" % (name, v))
    for name, v in zip(MMA_NAMES, mma_rates()):
        print("%-48s %7.2f cycles per product" % (name, v))
