"""GPU parity of dp_daq_quantize against the CPU oracle: codes, scales and row sums bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import to_dev_bf16

pytestmark = pytest.mark.gpu


def _run(x_bits, ldx=None, ldq=None, rowsum=True):
    M, K = x_bits.shape
    ldx = ldx or K
    ldq = ldq or K
    xb = np.zeros((M, ldx), np.uint16)
    xb[:, :K] = x_bits
    x = to_dev_bf16(xb)
    q = torch.full((M, ldq), 77, dtype=torch.int8, device="cuda")
    s_a = torch.empty(M, dtype=torch.float32, device="cuda")
    rs = torch.empty(M, dtype=torch.int32, device="cuda") if rowsum else None
    B.dp_daq_quantize(x, M, K, ldx, q, ldq, s_a, rs)
    torch.cuda.synchronize()
    return q.cpu().numpy(), s_a.cpu().numpy(), None if rs is None else rs.cpu().numpy()


@pytest.mark.parametrize("M,K", [(1, 128), (7, 1152), (256, 1152), (1000, 4608), (33, 2304),
                                 (19, 8), (5, 8200), (3, 65536)])
def test_daq_matches_oracle(M, K):
    x = synth.activations(synth.BASE_SEED, 3, 1, M, K, 1.0, n_out=max(1, K // 100))
    q, s_a, rs = _run(x, ldq=(K + 15) // 16 * 16)
    oq, osa, ors = oracle.daq(x)
    assert np.array_equal(s_a.view(np.uint32), osa.view(np.uint32))
    assert np.array_equal(q[:, :K], oq)
    assert np.array_equal(rs, ors)


def test_daq_edge_rows_and_pitch():
    K = 1152
    rng = np.random.default_rng(0)
    f = rng.standard_normal((12, K)).astype(np.float32)
    f[0] = 0.0                      # all-zero token
    f[1] = 2.0**-101                # below the threshold -> zero token
    f[2] = 2.0**-100                # at the threshold
    f[3] = 3.0e38                   # near the top of the bf16 range
    f[4] *= 1e-30
    f[5, :] = 0.0
    f[5, 700] = -5.0                # one-hot
    f[6] = np.where(np.arange(K) % 2 == 0, 0.5, 1.5) ; f[6, 0] = 127.0   # exact ties
    f[7] = np.where(np.arange(K) % 2 == 0, -2.5, 3.5) ; f[7, 1] = -127.0
    x = synth.f32_to_bf16_bits(f)
    q, s_a, rs = _run(x, ldx=K + 64, ldq=K + 128)
    oq, osa, ors = oracle.daq(x)
    assert np.array_equal(s_a.view(np.uint32), osa.view(np.uint32))
    assert np.array_equal(q[:, :K], oq) and np.all(q[:, K:] == 77)
    assert np.array_equal(rs, ors)
    q2, s2, none = _run(x, rowsum=False)
    assert none is None and np.array_equal(q2, oq)


def test_daq_empty_and_errors():
    x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((4, 128), dtype=torch.int8, device="cuda")
    s = torch.zeros(4, dtype=torch.float32, device="cuda")
    B.dp_daq_quantize(x, 0, 128, 128, q, 128, s)          # M = 0: no-op
    for args, code in [((x, 4, 100, 128, q, 128, s), B.DP_ERR_SHAPE),      # K % 8
                       ((x, 4, 128, 64, q, 128, s), B.DP_ERR_SHAPE),       # ldx < K
                       ((x, 4, 128, 128, q, 136, s), B.DP_ERR_ALIGN),      # ldq % 16
                       ((None, 4, 128, 128, q, 128, s), B.DP_ERR_INVALID_ARG)]:
        with pytest.raises(B.DiffproError) as e:
            B.dp_daq_quantize(*args)
        assert e.value.status == code
