"""ctypes binding of the benchmark's probe library (``include/distsim_bench.h``,
``libdistsim_bench.so``): integer-issue probes that measure the device's plain-integer peaks.
Measurement code only; the engine's library does not contain it."""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdistsim_bench.so")
EXPORTS = ("distsim_bench_int_issue_probe",)

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2306_08423_b200.build`")
_lib = C.CDLL(LIB_PATH)
_lib.distsim_bench_int_issue_probe.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                               C.POINTER(C.c_int64)]


def distsim_bench_int_issue_probe(blocks: int, iters: int, mode: int, d_sink, stream=None) -> int:
    """Enqueues the probe on the current device; returns the number of integer instructions it
    runs.  ``d_sink`` is a CUDA int64 tensor of at least one element (the caller's)."""
    import torch
    if not d_sink.is_cuda or d_sink.dtype != torch.int64 or d_sink.numel() < 1:
        raise ValueError("d_sink: need a CUDA int64 tensor")
    s = torch.cuda.current_stream() if stream is None else stream
    ops = C.c_int64(0)
    rc = _lib.distsim_bench_int_issue_probe(C.c_void_p(s.cuda_stream), mode, blocks, iters,
                                            C.c_void_p(d_sink.data_ptr()), C.byref(ops))
    if rc != 0:
        raise RuntimeError(f"distsim_bench_int_issue_probe failed ({rc})")
    return int(ops.value)
