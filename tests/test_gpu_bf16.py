"""GPU parity of the 16-bit pass-through layers (dp_weight.bits = 16: bf16 x bf16 -> fp32 -> bf16 on the
tensor cores) against the oracle's double-precision linear.

Tolerance. The oracle sums in double and rounds once; the tensor core accumulates K products in fp32
in an order of its own, so |y_gpu - exact| <= 2^-8 |exact| (the bf16 rounding, half an ulp, plus one
ulp of slack for a value pushed across a rounding boundary) + K * 2^-23 * sum_k |x w| (K fp32 additions
of magnitude at most the absolute sum, each within 2^-24 relative, with a factor 2 of margin for
truncating alignment inside the tensor core). Measured distances are 0 or 1 bf16 ulp."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import to_dev_bf16, bf16_to_np
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu
SEED = synth.BASE_SEED + 16


def _weights_bf16(layer, N, K):
    w8, s_w = synth.weights(SEED, layer, N, K, 8)
    return synth.f32_to_bf16_bits(w8.astype(np.float32) * s_w[:, None])


def _run(x_bits, w_bits, bias_bits, ldy=None):
    M, K = x_bits.shape
    N = w_bits.shape[0]
    wd = to_dev_bf16(w_bits)
    bd = None if bias_bits is None else to_dev_bf16(bias_bits)
    W = B.dp_weight(N, K, 16, 0, wd.data_ptr(), None, None if bd is None else bd.data_ptr())
    ldy = N if ldy is None else ldy
    y = torch.full((M, ldy), float("nan"), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dp_wq_linear(W, to_dev_bf16(x_bits), K, None, M, y, ldy, None, None, st, 0)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return bf16_to_np(y)


def _check(got, x, w, b):
    y, exact, mag = oracle.linear_bf16(x, w, b)
    gf = synth.bf16_bits_to_f32(got).astype(np.float64)
    K = x.shape[1]
    tol = np.abs(exact) * 2.0**-8 + K * 2.0**-23 * mag + 1e-30
    assert np.all(np.abs(gf - exact) <= tol), float(np.max(np.abs(gf - exact) / tol))
    d = bf16_ulp_dist(got, y)
    # where the output is not a near-total cancellation, the two roundings agree to an ulp
    big = np.abs(exact) > 2.0**-6 * mag
    assert d[big].max() <= 1 and (d[big] != 0).mean() < 0.05


@pytest.mark.parametrize("M,K,N", [(128, 128, 64), (200, 384, 192), (77, 1152, 384), (300, 256, 512),
                                   (1000, 4608, 1152), (16, 1152, 6912), (2048, 1152, 1152)])
def test_passthrough_layer_matches_double_precision_linear(M, K, N):
    """Every tile width (64, 128, 256), ragged and small M, short and long K, more tiles than SMs."""
    x = synth.activations(SEED, N % 7, 0, M, K, 1.0, n_out=max(1, K // 100))
    w = _weights_bf16(1, N, K)
    b = synth.bias(SEED, 1, N) if N != 192 else None
    _check(_run(x, w, b), x, w, b)


def test_passthrough_layer_output_pitch_and_unwritten_padding():
    M, K, N = 130, 256, 128
    x = synth.activations(SEED, 0, 0, M, K, 1.0, n_out=2)
    w = _weights_bf16(2, N, K)
    got = _run(x, w, None, ldy=N + 8)          # rows 16-byte but not 32-byte aligned: the narrow store form
    _check(got[:, :N], x, w, None)
    assert np.all(got[:, N:] == 0x7FC0)        # the padding columns keep the NaN fill


def test_plan_with_frozen_16_bit_layers_runs_end_to_end():
    """A bit plan that mixes 16-bit pass-through layers with 8/4/3-bit quantized ones, as the paper's
    best plans do (the most sensitive layers stay in 16-bit precision): Phase B over two steps."""
    from gpu_util import DevLayer
    table = [(256, 256, 128, 16), (256, 128, 256, 4), (16, 256, 128, 16), (256, 256, 192, 8), (256, 256, 128, 3)]
    devs, hosts, keep = [], [], []
    for l, (M, K, N, bits) in enumerate(table):
        b = synth.bias(SEED, l, N)
        if bits == 16:
            w = _weights_bf16(l, N, K)
            wd, bd = to_dev_bf16(w), to_dev_bf16(b)
            keep += [wd, bd]
            devs.append(B.dp_weight(N, K, 16, 0, wd.data_ptr(), None, bd.data_ptr()))
            hosts.append((w, None, b))
        else:
            w, s_w = synth.weights(SEED, l, N, K, bits)
            L = DevLayer(w, s_w, b, bits)
            keep.append(L)
            devs.append(L.w)
            hosts.append((w, s_w, b))
    plan = B.dp_plan_create(devs, [t[0] for t in table], B.DP_FLAG_GROUP_SMALL_M)
    try:
        kept = [3, 7]
        xs = [[synth.activations(SEED, l, t, M, K, synth.sigma_t(t, 10), n_out=2) for l, (M, K, N, _) in enumerate(table)]
              for t in kept]
        xd = [[to_dev_bf16(x) for x in row] for row in xs]
        ys = [[torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for (M, K, N, _) in table] for _ in kept]
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dp_plan_run(plan, kept, 0, B.ptr_array([t.data_ptr() for row in xd for t in row]),
                      B.ptr_array([t.data_ptr() for row in ys for t in row]), ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        for i in range(len(kept)):
            for l, (M, K, N, bits) in enumerate(table):
                w, s_w, b = hosts[l]
                got = bf16_to_np(ys[i][l])
                if bits == 16:
                    _check(got, xs[i][l], w, b)
                else:
                    ref = oracle.wq_linear(xs[i][l], oracle.pack(w, bits), s_w, b, bits)
                    assert bf16_ulp_dist(got, ref).max() <= 1
    finally:
        B.dp_plan_destroy(plan)


def test_passthrough_layer_argument_errors():
    w = torch.zeros((96, 128), dtype=torch.bfloat16, device="cuda")
    W = B.dp_weight(96, 128, 16, 0, w.data_ptr(), None, None)       # N % 64 != 0
    x = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((8, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(W, x, 128, None, 8, y, 96, None)
    assert e.value.status == B.DP_ERR_SHAPE
    W = B.dp_weight(128, 128, 16, 0, w.data_ptr(), None, None)
    sa = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(B.DiffproError) as e:                         # quantized activations make no sense here
        B.dp_wq_linear(W, x, 128, sa, 8, y, 128, None)
    assert e.value.status == B.DP_ERR_INVALID_ARG
