"""dp_wq_linear_static: the quantized linear for callers that may not allocate device memory.

Such callers (a custom-op slot of a runtime that owns all device memory, code running during a
stream capture, a loop that cannot afford an allocation's device stall) get the scratch from a
fixed array inside the library instead of a `workspace` argument. The result must be the one
dp_wq_linear gives with a caller-provided workspace, and both must be the CPU oracle's layer (so the
check does not rest on the library agreeing with itself). Calls in a row on different problems check
that the shared array, which keeps the previous call's contents, is fully re-initialised by each
call. This file is collected last so a failure here cannot mask any other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import DevLayer, to_dev_bf16, bf16_to_np
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu
SEED = synth.BASE_SEED + 9


def _both(M, K, N, bits, layer):
    x = synth.activations(SEED, layer, 0, M, K, 1.0, n_out=max(1, K // 100))
    w, s_w = synth.weights(SEED, layer, N, K, bits)
    b = synth.bias(SEED, layer, N)
    L = DevLayer(w, s_w, b, bits)
    xd = to_dev_bf16(x)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_ref = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, bits), dtype=torch.uint8, device="cuda")
    B.dp_wq_linear(L.w, xd, K, None, M, y_ref, N, ws, None, status)
    y_new = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.dp_wq_linear_static(L.w, xd, K, M, y_new, N, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    y_orc = oracle.wq_linear(x, oracle.pack(w, bits), s_w, b, bits)
    return bf16_to_np(y_new), bf16_to_np(y_ref), y_orc


def test_static_scratch_matches_workspace_variant_on_calls_in_a_row():
    # first call: a larger problem fills much of the array; the following, smaller ones with other
    # widths must not see anything of it
    for (M, K, N, bits, layer) in [(1000, 1152, 384, 4, 0), (300, 256, 128, 8, 1), (16, 1152, 96, 3, 2)]:
        got, ref, orc = _both(M, K, N, bits, layer)
        assert not np.any(got == 0x7FC0), "output not fully written"
        assert bf16_ulp_dist(got, ref).max() <= 1
        assert np.array_equal(got, ref)
        d = bf16_ulp_dist(got, orc)       # the oracle's layer: within 1 bf16 ulp, almost all equal
        assert d.max() <= 1 and (d != 0).mean() < 1e-3


def test_static_scratch_rejects_oversized_problems():
    K, N = 4608, 128
    w, s_w = synth.weights(SEED, 3, N, K, 8)
    L = DevLayer(w, s_w, None, 8)
    M = 4096                                  # 4096 x 4608 int8 codes > 10 MiB
    assert B.dp_wq_linear_workspace(M, N, K, 8) > B.DP_STATIC_SCRATCH_BYTES
    x = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear_static(L.w, x, K, M, y, N)
    assert e.value.status == B.DP_ERR_WORKSPACE and "scratch" in str(e.value)
