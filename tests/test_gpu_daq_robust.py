"""GPU parity of dp_daq_quantize_robust (Eq. "daq" with its percentile clip, nearest-rank reading, and
a-bit codes) against the CPU oracle: codes, scales and row sums bit-exact; and of the two-call
pipeline robust DAQ -> dp_wq_linear on quantized activations against the oracle's composition."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import DevLayer, to_dev_bf16, bf16_to_np
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu


def _run(x_bits, rank, bits, ldx=None, ldq=None, rowsum=True):
    M, K = x_bits.shape
    ldx, ldq = ldx or K, ldq or (K + 15) // 16 * 16
    xb = np.zeros((M, ldx), np.uint16)
    xb[:, :K] = x_bits
    x = to_dev_bf16(xb)
    q = torch.full((M, ldq), 77, dtype=torch.int8, device="cuda")
    s_a = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
    rs = torch.full((M,), -5, dtype=torch.int32, device="cuda") if rowsum else None
    B.dp_daq_quantize_robust(x, M, K, ldx, q, ldq, s_a, rank, bits, rs)
    torch.cuda.synchronize()
    return q.cpu().numpy(), s_a.cpu().numpy(), None if rs is None else rs.cpu().numpy()


def _same(got, x, rank, bits):
    q, s_a, rs = got
    oq, osa, ors = oracle.daq_robust(x, rank, bits)
    K = x.shape[1]
    assert np.array_equal(s_a.view(np.uint32), osa.view(np.uint32)), "scales differ"
    assert np.array_equal(q[:, :K], oq), "codes differ"
    assert (q[:, K:] == 77).all(), "padding touched"
    if rs is not None:
        assert np.array_equal(rs, ors)


@pytest.mark.parametrize("M,K", [(1, 128), (7, 1152), (300, 1152), (260, 4608), (33, 2304), (19, 8), (5, 1160)])
@pytest.mark.parametrize("rank,bits", [(1, 8), (2, 8), (5, 8), (12, 6), (3, 4), (2, 2)])
def test_matches_oracle(M, K, rank, bits):
    rank = min(rank, K)
    x = synth.activations(synth.BASE_SEED, 5, 2, M, K, 1.3, n_out=max(1, K // 100))
    _same(_run(x, rank, bits), x, rank, bits)


def test_percentile_of_the_paper_on_the_benchmark_shapes():
    """p = 99.9: rank 2 at K = 1152, rank 5 at K = 4608 (outlier channels x20 make the clip bite)."""
    for K in (1152, 4608):
        rank = B.dp_clip_rank(99900, K)
        assert rank == oracle.clip_rank("99.9", K) == (2 if K == 1152 else 5)
        x = synth.activations(synth.BASE_SEED, 1, 3, 512, K, 1.0, n_out=K // 100)
        got = _run(x, rank, 8)
        _same(got, x, rank, 8)
        assert (np.abs(got[0][:, :K]) == 127).sum(axis=1).min() >= rank  # the clipped values sit on the extremes


def test_repeats_sparse_rows_and_pitches():
    K = 1152
    rng = np.random.default_rng(3)
    x = synth.f32_to_bf16_bits(rng.standard_normal((40, K)).astype(np.float32))
    x[0, :] = x[0, 0]                                  # constant row
    x[1, :] = 0                                        # zero row
    x[2, :] = 0
    x[2, 17] = 0x4040                                  # one non-zero value: rank 2 threshold is zero
    x[3, :100] = x[3, 100] | 0x8000                    # 101 equal magnitudes, mixed signs
    x[4, :] = synth.f32_to_bf16_bits((rng.integers(-3, 4, K)).astype(np.float32))  # heavy ties
    x[5, :] = 0x0001                                   # smallest subnormal everywhere: below 2^-100
    for rank, bits in ((1, 8), (2, 8), (7, 5), (64, 8)):
        _same(_run(x, rank, bits, ldx=K + 8, ldq=K + 32), x, rank, bits)


def test_pipeline_with_the_linear_matches_the_oracle_composition():
    """Robust DAQ's codes and scales fed to dp_wq_linear as quantized activations (tensor-core and
    small-M kernels): int32 sums and outputs as the oracle composes them."""
    for M, K, N, wbits, flags in ((300, 1152, 384, 4, B.DP_FLAG_FORCE_MMA), (8, 1152, 96, 3, B.DP_FLAG_FORCE_SIMT)):
        x = synth.activations(synth.BASE_SEED, 6, 4, M, K, 1.0, n_out=11)
        w, s_w = synth.weights(synth.BASE_SEED, 6, N, K, wbits)
        b = synth.bias(synth.BASE_SEED, 6, N)
        rank = B.dp_clip_rank(99900, K)
        oq, osa, _ = oracle.daq_robust(x, rank, 6)
        ref = oracle.epilogue(oracle.gemm_i32(oq, w), osa, s_w, b)
        L = DevLayer(w, s_w, b, wbits)
        xd = to_dev_bf16(x)
        q = torch.empty((M, K), dtype=torch.int8, device="cuda")
        s_a = torch.empty(M, dtype=torch.float32, device="cuda")
        B.dp_daq_quantize_robust(xd, M, K, K, q, K, s_a, rank, 6)
        y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, wbits, flags), dtype=torch.uint8, device="cuda")
        B.dp_wq_linear(L.w, q, K, s_a, M, y, N, ws, None, status, flags)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert bf16_ulp_dist(bf16_to_np(y), ref).max() <= 1


def test_argument_errors():
    x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((4, 128), dtype=torch.int8, device="cuda")
    s = torch.zeros(4, dtype=torch.float32, device="cuda")
    for rank, bits, status in ((0, 8, B.DP_ERR_INVALID_ARG), (65, 8, B.DP_ERR_INVALID_ARG), (2, 9, B.DP_ERR_BITS),
                               (2, 1, B.DP_ERR_BITS)):
        with pytest.raises(B.DiffproError) as e:
            B.dp_daq_quantize_robust(x, 4, 128, 128, q, 128, s, rank, bits)
        assert e.value.status == status
    with pytest.raises(B.DiffproError) as e:
        B.dp_daq_quantize_robust(x, 4, 8192, 8192, q, 8192, s, 2, 8)
    assert e.value.status == B.DP_ERR_SHAPE
