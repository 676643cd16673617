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
from gpu_util import bf16_to_np, to_dev_bf16
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


def _run_layer(W, x_bits_or_dev, M, K, N, bits, flags=0):
    x = x_bits_or_dev if torch.is_tensor(x_bits_or_dev) else to_dev_bf16(x_bits_or_dev)
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, bits, flags), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dp_wq_linear(W.w, x, K, None, M, y, N, ws, None, status, flags)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return y


def test_c1_single_proj_linear_whole_output():
    """M = 256 tokens, 1152 -> 1152, int8 weights, 8 outlier channels: every output element."""
    seed, layer, M, K, N, bits = synth.BASE_SEED + 1, 0, 256, 1152, 1152, 8
    x = synth.activations(seed, layer, 0, M, K, 1.0, n_out=8)
    y = _run_layer(DevWeights(seed, layer, N, K, bits), x, M, K, N, bits)
    _check_rows(y, x, list(range(M)), seed, layer, N, K, bits, "c1")


def test_c2_fc1_4bit_whole_output():
    """M = 2048, 1152 -> 4608 at 4 bits, 1 % outlier channels: every output element."""
    seed, layer, M, K, N, bits = synth.BASE_SEED + 2, 0, 2048, 1152, 4608, 4
    x = synth.activations(seed, layer, 0, M, K, 1.0, n_out=K // 100)
    y = _run_layer(DevWeights(seed, layer, N, K, bits), x, M, K, N, bits)
    _check_rows(y, x, list(range(M)), seed, layer, N, K, bits, "c2")


def test_c3_block_at_m4096_with_gelu_input_sampled_rows():
    """One block's linears at M = 4096 (adaLN M = 16), bits from {4, 8}; fc2 reads GELU(N(0,1)):
    non-negative, heavy-tailed, the case where absmax scaling wastes half the code range."""
    seed = synth.BASE_SEED + 3
    table = [("qkv", 4096, 1152, 3456), ("proj", 4096, 1152, 1152), ("fc1", 4096, 1152, 4608),
             ("fc2", 4096, 4608, 1152), ("adaln", 16, 1152, 6912)]
    bits = synth.bit_plan(seed, len(table), (4, 8))
    rng = np.random.default_rng(3)
    for l, (name, M, K, N) in enumerate(table):
        x = (synth.gelu_activations(seed, l, 0, M, K) if name == "fc2"
             else synth.activations(seed, l, 0, M, K, 1.0, n_out=K // 100))
        y = _run_layer(DevWeights(seed, l, N, K, bits[l]), x, M, K, N, bits[l])
        rows = _sample_rows(M, rng, n=12)
        _check_rows(y, x[rows], rows, seed, l, N, K, bits[l], ("c3", name, bits[l]))


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
