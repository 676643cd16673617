"""ctypes binding of libdpprobe.so: measurement probes kept outside the product library
(include/diffpro_probe.h)."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdpprobe.so")
_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with python -m paper_2511_11446_b200.build")
        _lib = C.CDLL(LIB_PATH)
        _lib.dp_probe_mma_i8.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    return _lib


def dp_probe_mma_i8(ctas, iters, tile_n=256, device_status=None, stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    st = lib().dp_probe_mma_i8(ctas, iters, tile_n, None if device_status is None else C.c_void_p(device_status.data_ptr()),
                               C.c_void_p(s.cuda_stream))
    if st != 0:
        raise RuntimeError(f"dp_probe_mma_i8 failed with status {st}")
