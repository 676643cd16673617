"""dp_ln_modulate_daq against the oracle: int8 codes and token scales bit for bit (both sides take the
statistics in double from exact sums and run one fp32 sequence), alone and in front of dp_wq_linear."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import DevLayer, to_dev_bf16, bf16_to_np

pytestmark = pytest.mark.gpu
EPS = 1e-6


def _inputs(M, K, seed, rps):
    s = synth.BASE_SEED + 700 + seed
    x = synth.activations(s, 0, 0, M, K, 1.0, n_out=max(1, K // 100))
    rng = np.random.default_rng(s)
    S = -(-M // rps)
    shift = synth.f32_to_bf16_bits(rng.normal(0, 0.3, (S, K)).astype(np.float32))
    scale = synth.f32_to_bf16_bits(rng.normal(0, 0.3, (S, K)).astype(np.float32))
    return x, shift, scale


def _run(x, shift, scale, rps, ldq=None):
    M, K = x.shape
    ldq = K if ldq is None else ldq
    xd = to_dev_bf16(x)
    shd = None if shift is None else to_dev_bf16(shift)
    scd = None if scale is None else to_dev_bf16(scale)
    q = torch.full((M, ldq), 99, dtype=torch.int8, device="cuda")
    sa = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
    B.dp_ln_modulate_daq(xd, M, K, K, shd, scd, rps, EPS, q, ldq, sa)
    torch.cuda.synchronize()
    return q.cpu().numpy(), sa.cpu().numpy(), (q, sa)


@pytest.mark.parametrize("M,K,rps", [(2048, 1152, 256), (300, 1152, 77), (9, 64, 4), (1000, 4608, 256), (37, 1280, 1)])
@pytest.mark.parametrize("mod", [True, False])
def test_codes_and_scales_match_the_oracle(M, K, rps, mod):
    x, shift, scale = _inputs(M, K, K % 97 + M % 13, rps)
    if not mod:
        shift = scale = None
    q, sa, _ = _run(x, shift, scale, rps)
    qo, so = oracle.ln_modulate_daq(x, shift, scale, rps, EPS)
    assert np.array_equal(sa.view(np.uint32), so.view(np.uint32)), "token scales differ"
    bad = np.argwhere(q != qo)
    assert bad.size == 0, (len(bad), bad[:5].tolist())


def test_constant_and_zero_tokens_and_pitch():
    M, K = 16, 256
    x, shift, scale = _inputs(M, K, 5, 8)
    x[3] = synth.f32_to_bf16_bits(np.array([2.5], np.float32))[0]   # zero variance: h = shift
    x[7] = 0
    q, sa, _ = _run(x, shift, scale, 8, ldq=K + 32)
    qo, so = oracle.ln_modulate_daq(x, shift, scale, 8, EPS)
    assert np.array_equal(sa.view(np.uint32), so.view(np.uint32))
    assert np.array_equal(q[:, :K], qo) and np.all(q[:, K:] == 99)
    q2, sa2, _ = _run(x, None, None, 1)
    assert not q2[3].any() and sa2[3] == 0.0 and not q2[7].any() and sa2[7] == 0.0


def test_feeds_the_quantized_linear():
    """LayerNorm + modulate + DAQ, then dp_wq_linear on the codes: equal to the oracle's composition."""
    M, K, N, bits, rps = 512, 1152, 384, 4, 256
    x, shift, scale = _inputs(M, K, 9, rps)
    w, s_w = synth.weights(synth.BASE_SEED + 9, 0, N, K, bits)
    b = synth.bias(synth.BASE_SEED + 9, 0, N)
    L = DevLayer(w, s_w, b, bits)
    _, _, (qd, sad) = _run(x, shift, scale, rps)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    flags = B.DP_FLAG_FORCE_MMA
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, bits, flags), dtype=torch.uint8, device="cuda")
    B.dp_wq_linear(L.w, qd, K, sad, M, y, N, ws, None, st, flags)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    qo, so = oracle.ln_modulate_daq(x, shift, scale, rps, EPS)
    acc = oracle.gemm_i32(qo, w)
    want = oracle.epilogue(acc, so, s_w, b)
    assert np.array_equal(bf16_to_np(y), want)


def test_argument_errors():
    x = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((8, 64), dtype=torch.int8, device="cuda")
    sa = torch.zeros(8, device="cuda")
    v = torch.zeros((1, 64), dtype=torch.bfloat16, device="cuda")
    for args in ((x, 8, 60, 64, None, None, 1, EPS, q, 64, sa),          # K not a multiple of 8
                 (x, 8, 64, 64, v, None, 8, EPS, q, 64, sa),             # shift without scale
                 (x, 8, 64, 64, v, v, 0, EPS, q, 64, sa),                # rows_per_sample
                 (x, 8, 64, 64, None, None, 1, EPS, q, 48, sa)):         # ldq < K
        with pytest.raises(B.DiffproError):
            B.dp_ln_modulate_daq(*args)
