"""Pins for the oracle's linear with the residual (and adaLN gate) taken into the epilogue."""
from fractions import Fraction

import numpy as np

import oracle
from paper_2511_11446_b200 import synth
from helpers import f32_frac, round_frac_to_f32
from test_oracle_pack_gemm import _bf16_rne_bits


def _case(M, K, N, bits, seed):
    s = synth.BASE_SEED + seed
    x = synth.activations(s, 0, 0, M, K, 1.0, n_out=2)
    w, s_w = synth.weights(s, 0, N, K, bits)
    b = synth.bias(s, 0, N)
    res = synth.activations(s, 1, 0, M, N, 1.0, n_out=0)
    return x, w, s_w, b, res


def test_exact_sequence_with_and_without_gate():
    """lin = RN(float(acc) * RN(s_a * s_w) + bias); v = RN(gate * lin + res) or RN(lin + res);
    y = bf16_RNE(v): evaluated in exact rationals, compared for equality (an epilogue that rounded lin
    to bf16 before adding, or added the residual before the gate, lands elsewhere)."""
    M, K, N, bits, rpg = 6, 256, 5, 4, 4
    x, w, s_w, b, res = _case(M, K, N, bits, 40)
    gate = synth.f32_to_bf16_bits(np.array([[0.5, -1.25, 2.0, 0.0, 1.0], [1.5, 0.75, -0.5, 3.0, 0.125]], np.float32))
    q, s_a, _ = oracle.daq(x)
    acc = oracle.gemm_i32(q, w)
    bf, rf, gf = (synth.bf16_bits_to_f32(t) for t in (b, res, gate))
    for g in (None, gate):
        y = oracle.wq_linear_residual(x, oracle.pack(w, bits), s_w, b, bits, res, g, rpg)
        n_other = 0
        for m in range(M):
            for n in range(N):
                t = f32_frac(round_frac_to_f32(Fraction(int(acc[m, n]))))
                sc = f32_frac(round_frac_to_f32(f32_frac(s_a[m]) * f32_frac(s_w[n])))
                lin = f32_frac(round_frac_to_f32(t * sc + f32_frac(bf[n])))
                r = f32_frac(rf[m, n])
                v = round_frac_to_f32(f32_frac(gf[m // rpg, n]) * lin + r) if g is not None else round_frac_to_f32(lin + r)
                assert int(y[m, n]) == _bf16_rne_bits(v), (m, n)
                lin16 = f32_frac(synth.bf16_bits_to_f32(np.array([_bf16_rne_bits(round_frac_to_f32(lin))], np.uint16))[0])
                alt = round_frac_to_f32((f32_frac(gf[m // rpg, n]) if g is not None else 1) * lin16 + r)
                n_other += _bf16_rne_bits(alt) != int(y[m, n])
        assert n_other >= 1          # rounding lin to bf16 first is a different function on these cases


def test_reduces_to_the_plain_layer():
    """res = 0 without a gate is orc_wq_linear; gate = 1 with any res equals the ungated form."""
    M, K, N, bits = 9, 128, 16, 8
    x, w, s_w, b, res = _case(M, K, N, bits, 41)
    pw = oracle.pack(w, bits)
    zero = np.zeros((M, N), np.uint16)
    assert np.array_equal(oracle.wq_linear_residual(x, pw, s_w, b, bits, zero), oracle.wq_linear(x, pw, s_w, b, bits))
    one = synth.f32_to_bf16_bits(np.ones((3, N), np.float32))
    assert np.array_equal(oracle.wq_linear_residual(x, pw, s_w, b, bits, res, one, 4),
                          oracle.wq_linear_residual(x, pw, s_w, b, bits, res))
    # gate rows follow m // rows_per_gate: a gate that is 0 on the second sample leaves res there
    g = synth.f32_to_bf16_bits(np.stack([np.ones(N), np.zeros(N), np.ones(N)]).astype(np.float32))
    y = oracle.wq_linear_residual(x, pw, s_w, b, bits, res, g, 4)
    assert np.array_equal(y[4:8], res[4:8])
