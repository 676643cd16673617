"""ctypes binding of libdpsynth.so: the CUDA implementation of the seeded input generators,
bit-identical to ``synth`` (numpy). Used for inputs too large to generate on the host."""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import synth

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdpsynth.so")
_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2511_11446_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.dps_activations.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_uint64,
                                      C.c_float, C.c_void_p, C.c_void_p]
        L.dps_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_uint64, C.c_int,
                                  C.c_void_p]
        _lib = L
    return _lib


def _s():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def activations(seed, layer, t, M, K, sigma=1.0, n_out=0, factor=20.0, out=None):
    """bf16 tensor [M,K] on the current device; same values as synth.activations."""
    cs = torch.from_numpy(synth.outlier_colscale(seed, layer, t, K, n_out, factor)).cuda()
    x = torch.empty((M, K), dtype=torch.bfloat16, device="cuda") if out is None else out
    rc = lib().dps_activations(x.data_ptr(), M, K, K, synth.stream_key(seed, synth.KIND_ACT, layer, t),
                               float(sigma), cs.data_ptr(), _s())
    if rc:
        raise RuntimeError(f"dps_activations: CUDA error {rc}")
    return x


def weights(seed, layer, N, K, bits):
    """(w int8 [N,K], s_w fp32 [N]) on the current device; same values as synth.weights."""
    w = torch.empty((N, K), dtype=torch.int8, device="cuda")
    s_w = torch.empty(N, dtype=torch.float32, device="cuda")
    rc = lib().dps_weights(w.data_ptr(), s_w.data_ptr(), N, K,
                           synth.stream_key(seed, synth.KIND_WEIGHT, layer, 0), bits, _s())
    if rc:
        raise RuntimeError(f"dps_weights: CUDA error {rc}")
    return w, s_w
