"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot redo a whole 45 TOP plan run, but DAQ and the linear are row-wise: for sampled
token rows it recomputes complete output rows one by one (all N channels) from inputs regenerated
on the host from the seed, and those must match what the GPU path wrote. Same tolerance as the
small cases: bf16 outputs within 1 ulp (the fp32 sequences are identical, so almost all are equal).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth, synth_cuda
from paper_2511_11446_b200.workloads import DitStack, DevWeights
from gpu_util import bf16_to_np
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu


def _sample_rows(M, rng, n=6):
    """Rows from the first, last and interior 128-token tiles (ragged ends included)."""
    fixed = {0, M - 1, min(M - 1, 127), min(M - 1, 128), M // 2}
    while len(fixed) < min(M, n + 4):
        fixed.add(int(rng.integers(0, M)))
    return sorted(fixed)


def _check_rows(y_dev, x_rows, rows, seed, layer, N, K, bits, what):
    w, s_w = synth.weights(seed, layer, N, K, bits)
    b = synth.bias(seed, layer, N)
    ref = oracle.wq_linear(x_rows, oracle.pack(w, bits), s_w, b, bits)
    got = bf16_to_np(y_dev[torch.tensor(rows, device="cuda")])
    d = bf16_ulp_dist(got, ref)
    assert d.max() <= 1, (what, int(d.max()))
    assert (d != 0).mean() < 1e-3, what


def test_c4_plan_run_as_benchmarked_sampled_rows():
    """The benchmark's plan (140 layers, M = 2048 / adaLN M = 8, mixed {3,4,8} bits, autotuned variants,
    grouped adaLN launch), one retained timestep: sampled rows of layers covering every shape and
    bit-width, and every adaLN layer of the first blocks."""
    stack = DitStack(resident_steps=1)  # bench.py's defaults: DP_FLAG_AUTOTUNE | DP_FLAG_GROUP_SMALL_M
    stack.run(1)
    torch.cuda.synchronize()
    assert int(stack.status.item()) == 0
    t = stack.kept[0]
    rng = np.random.default_rng(7)
    seen, chosen = set(), []
    for l, (name, M, K, N) in enumerate(stack.table):
        key = (name, stack.bits[l], B.dp_plan_layer_variant(stack.plan, l)["unpack_first"])
        if key not in seen or (M <= 32 and l < 15):
            seen.add(key)
            chosen.append(l)
    assert len(chosen) >= 15
    for l in chosen:
        name, M, K, N = stack.table[l]
        rows = _sample_rows(M, rng)
        x_rows = stack.host_input_rows(l, t, rows)
        _check_rows(stack.y[l], x_rows, rows, stack.seed, l, N, K, stack.bits[l],
                    (l, name, stack.bits[l], B.dp_plan_layer_variant(stack.plan, l)))


@pytest.mark.parametrize("name,K,N,M,bits", [("qkv", 1152, 3456, 32768, 4), ("proj", 1152, 1152, 32768, 3),
                                             ("fc1", 1152, 4608, 32768, 8), ("fc2", 4608, 1152, 32768, 4),
                                             ("fc2", 4608, 1152, 32768, 3), ("adaln", 1152, 6912, 32, 3),
                                             ("adaln", 1152, 6912, 32, 8)])
def test_c5_large_m_layers_sampled_rows(name, K, N, M, bits):
    """M = 32768 (batch 32 at 512 px; adaLN M = 32), default dispatch of dp_wq_linear."""
    seed, layer = synth.BASE_SEED + 5, 3
    n_out = max(1, K // 100)
    W = DevWeights(seed, layer, N, K, bits)
    x = synth_cuda.activations(seed, layer, 0, M, K, 1.0, n_out=n_out)
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, bits, 0), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dp_wq_linear(W.w, x, K, None, M, y, N, ws, None, status, 0)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = _sample_rows(M, np.random.default_rng(M + N + bits), n=10)
    x_rows = synth.activations(seed, layer, 0, M, K, 1.0, n_out=n_out, rows=rows)
    _check_rows(y, x_rows, rows, seed, layer, N, K, bits, (name, M, bits))
    # every row was written (no NaN sentinel left) -- a property that holds at any size
    assert not torch.isnan(y.float()).any()
