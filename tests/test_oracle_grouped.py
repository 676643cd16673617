"""Pins for the oracle's layer with group-wise weight scales (and zero-points)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_11446_b200 import synth
from helpers import f32_frac, round_frac_to_f32, bf16_ulp_dist
from test_oracle_pack_gemm import _bf16_rne_bits


def _case(M, K, N, bits, g, seed, zeros=False):
    rng = np.random.default_rng(seed)
    x = synth.activations(synth.BASE_SEED + seed, 0, 0, M, K, 1.0, n_out=max(1, K // 100))
    half = 1 << (bits - 1)
    w = rng.integers(-half, half, size=(N, K)).astype(np.int8)
    s_w = (np.abs(rng.standard_normal((N, K // g))) * 1e-2 + 1e-4).astype(np.float32)
    b = synth.bias(synth.BASE_SEED + seed, 0, N)
    z = rng.integers(0, 1 << bits, size=(N, K // g)).astype(np.uint8) if zeros else None
    return x, w, s_w, b, z


@pytest.mark.parametrize("bits,g,zeros", [(8, 32, False), (4, 64, False), (3, 32, True), (4, 128, True), (8, 96, False)])
def test_exact_fp32_sequence_in_rationals(bits, g, zeros):
    """Every output equals the defined sequence evaluated in exact rationals with one rounding per
    operation: acc_G exact; t <- RN(float(acc_G) * s + t) over the groups in order (float(acc_G) is
    itself RN of the integer); y = bf16_RNE(RN(t * s_a + bias)). A different group order, an unfused
    multiply-add or a per-channel scale would not reproduce these bits."""
    M, K, N = 5, 384, 6
    x, w, s_w, b, z = _case(M, K, N, bits, g, 100 + bits + g, zeros)
    y = oracle.wq_linear_grouped(x, oracle.pack(w, bits), s_w, b, bits, g, z)
    q, s_a, _ = oracle.daq(x)
    half = 1 << (bits - 1)
    bf = synth.bf16_bits_to_f32(b)
    for m in range(M):
        for n in range(N):
            t = Fraction(0)
            for G in range(K // g):
                zz = int(z[n, G]) if z is not None else half
                acc = sum(int(q[m, k]) * (int(w[n, k]) + half - zz) for k in range(G * g, (G + 1) * g))
                a32 = f32_frac(round_frac_to_f32(Fraction(acc)))
                t = f32_frac(round_frac_to_f32(a32 * f32_frac(s_w[n, G]) + t))
            y32 = round_frac_to_f32(t * f32_frac(s_a[m]) + f32_frac(bf[n]))
            assert int(y[m, n]) == _bf16_rne_bits(y32), (m, n)


def test_one_group_equal_scales_and_real_valued_accuracy():
    """(i) With one scale repeated over the groups the layer approximates the per-channel layer (same
    real-valued result, other roundings): within a few fp32 roundings of it. (ii) Against the
    real-valued linear of the dequantized weights the only errors are the activation rounding
    (<= s_a/2 per element) and the output rounding."""
    M, K, N, bits, g = 16, 512, 24, 4, 64
    x, w, s_w, b, _ = _case(M, K, N, bits, g, 7)
    s1 = np.repeat(s_w[:, :1], K // g, axis=1).copy()
    y = oracle.wq_linear_grouped(x, oracle.pack(w, bits), s1, b, bits, g)
    y_pc = oracle.wq_linear(x, oracle.pack(w, bits), s1[:, 0].copy(), b, bits)
    assert bf16_ulp_dist(y, y_pc).max() <= 1
    y = oracle.wq_linear_grouped(x, oracle.pack(w, bits), s_w, b, bits, g)
    q, s_a, _ = oracle.daq(x)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    wf = w.astype(np.float64) * np.repeat(s_w.astype(np.float64), g, axis=1)
    ref = xf @ wf.T + synth.bf16_bits_to_f32(b).astype(np.float64)[None, :]
    bound = (0.5 + 2.0**-15) * s_a.astype(np.float64)[:, None] * np.abs(wf).sum(axis=1)[None, :]
    got = synth.bf16_bits_to_f32(y).astype(np.float64)
    assert np.all(np.abs(got - ref) <= bound + np.abs(ref) * 2.0**-7 + 1e-6)


def test_zero_points_shift_the_codes_and_one_hot_tokens_pick_weights():
    """z = 2^(b-1) is the symmetric layer; a one-hot token (value 1 at k0 -> q = 127) returns
    127 * s_a * s_w[n][G(k0)] * (u[n,k0] - z[n][G(k0)]): catches a wrong group index, a sign error on
    z, or codes taken as signed when z is given."""
    M, K, N, bits, g = 3, 256, 10, 4, 32
    x, w, s_w, _, z = _case(M, K, N, bits, g, 9, zeros=True)
    half = 1 << (bits - 1)
    zsym = np.full((N, K // g), half, np.uint8)
    assert np.array_equal(oracle.wq_linear_grouped(x, oracle.pack(w, bits), s_w, None, bits, g, zsym),
                          oracle.wq_linear_grouped(x, oracle.pack(w, bits), s_w, None, bits, g, None))
    k0 = 77
    oh = np.zeros((1, K), np.float32)
    oh[0, k0] = 1.0
    xo = synth.f32_to_bf16_bits(oh)
    y = synth.bf16_bits_to_f32(oracle.wq_linear_grouped(xo, oracle.pack(w, bits), s_w, None, bits, g, z))[0]
    G = k0 // g
    want = (127.0 * (w[:, k0].astype(np.float64) + half - z[:, G])) * s_w[:, G].astype(np.float64) * (1.0 / 127.0)
    assert np.all(np.abs(y - want) <= np.abs(want) * 2.0**-7 + 1e-12)
