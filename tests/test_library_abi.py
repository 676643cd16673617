"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, and
its host-side helpers and argument checks behave. No kernel is launched."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2511_11446_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_exports_match_header():
    hdr = open(os.path.join(ROOT, "include", "diffpro.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(dp_[a-z0-9_]+)\s*\(", hdr))
    assert declared == set(B.EXPORTS)
    L = B.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert B.dp_version() >= 1
    assert L.dp_status_string(B.DP_ERR_TIMEOUT).decode() == "DP_ERR_TIMEOUT"


def test_probe_library_exports_its_header():
    """The measurement probes live in a library of their own, outside the product ABI."""
    from paper_2511_11446_b200 import probe
    hdr = open(os.path.join(ROOT, "include", "diffpro_probe.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(dp_[a-z0-9_]+)\s*\(", hdr))
    assert declared == {"dp_probe_mma_i8"}
    for name in declared:
        assert getattr(probe.lib(), name) is not None
        assert not hasattr(B.lib(), name)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_host_packer_agrees_with_oracle_codec(bits):
    rng = np.random.default_rng(bits)
    half = 1 << (bits - 1)
    w = rng.integers(-half, half, size=(33, 1152)).astype(np.int8)
    mine = B.dp_pack_weights_host(w, bits)
    assert np.array_equal(mine.view(np.uint8).ravel(), oracle.pack(w, bits).view(np.uint8).ravel())
    assert np.array_equal(oracle.unpack(mine, 1152, bits), w)
    if bits != 8:
        w[5, 77] = half
        with pytest.raises(B.DiffproError) as e:
            B.dp_pack_weights_host(w, bits)
        assert e.value.status == B.DP_ERR_INVALID_ARG


def test_argument_errors_detected_before_any_cuda_call():
    import ctypes as C
    L = B.lib()
    assert L.dp_daq_quantize(None, 4, 128, 128, None, 128, None, None, None) == B.DP_ERR_INVALID_ARG
    assert L.dp_daq_quantize(None, 4, 100, 128, None, 128, None, None, None) == B.DP_ERR_SHAPE
    assert L.dp_daq_quantize(None, 0, 128, 128, None, 128, None, None, None) == B.DP_OK
    assert B.dp_wq_linear_workspace(2048, 4608, 1152, 4) >= 2048 * 1152 + 4 * 2048
    assert B.dp_wq_linear_workspace(16, 6912, 1152, 4) == 256
    w = B.dp_weight(128, 100, 8, 0, 16, 16, None)
    assert L.dp_wq_linear(C.byref(w), None, 0, None, 0, None, 0, None, 0, None, None, 0, None) == B.DP_ERR_SHAPE
    w = B.dp_weight(128, 128, 6, 0, 16, 16, None)
    assert L.dp_wq_linear(C.byref(w), None, 0, None, 0, None, 0, None, 0, None, None, 0, None) == B.DP_ERR_BITS
    assert b"bits" in L.dp_last_error()
