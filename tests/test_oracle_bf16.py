"""Pins for the oracle's pass-through linear of 16-bit layers (y = x . W^T + bias on bf16 inputs)."""
from fractions import Fraction

import numpy as np
import torch

import oracle
from paper_2511_11446_b200 import synth


def _bf16(a):
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def test_against_numpy_float64_matmul_and_exact_rationals():
    rng = np.random.default_rng(16)
    M, K, N = 9, 384, 13
    x, w, b = _bf16(rng.standard_normal((M, K))), _bf16(rng.standard_normal((N, K)) * 0.05), _bf16(rng.standard_normal(N))
    y, exact, mag = oracle.linear_bf16(x, w, b)
    xf, wf, bf = (synth.bf16_bits_to_f32(t).astype(np.float64) for t in (x, w, b))
    ref = xf @ wf.T + bf[None, :]                       # library routine, float64
    assert np.allclose(exact, ref, rtol=0, atol=1e-12 * np.abs(xf).sum())
    assert np.allclose(mag, np.abs(xf) @ np.abs(wf).T, rtol=1e-12)
    # a few elements in exact rationals, rounded once to bf16 (ties to even)
    for (m, n) in [(0, 0), (3, 7), (8, 12)]:
        s = sum(Fraction(float(xf[m, k])) * Fraction(float(wf[n, k])) for k in range(K)) + Fraction(float(bf[n]))
        assert abs(Fraction(float(exact[m, n])) - s) <= abs(s) * Fraction(1, 2**45)
        cands = sorted({int(y[m, n]) - 1, int(y[m, n]), int(y[m, n]) + 1})
        vals = [(abs(Fraction(float(synth.bf16_bits_to_f32(np.array([c], np.uint16))[0])) - s), c & 1, c) for c in cands]
        assert min(vals)[2] == int(y[m, n])
    # without bias
    y0, e0, _ = oracle.linear_bf16(x, w, None)
    assert np.allclose(e0, xf @ wf.T, rtol=0, atol=1e-12 * np.abs(xf).sum())


def test_structure_identity_and_one_hot():
    K = 128
    rng = np.random.default_rng(3)
    x = _bf16(rng.standard_normal((5, K)))
    eye = _bf16(np.eye(K, dtype=np.float32))
    y, _, _ = oracle.linear_bf16(x, eye, None)
    assert np.array_equal(y, x)                          # W = I reproduces x (transposed operand would not for W != W^T)
    w = _bf16(rng.standard_normal((7, K)))
    oh = _bf16(np.eye(K, dtype=np.float32)[37:38] * 2.0)
    y, _, _ = oracle.linear_bf16(oh, w, None)
    assert np.array_equal(synth.bf16_bits_to_f32(y)[0], 2.0 * synth.bf16_bits_to_f32(w)[:, 37])


def test_final_rounding_is_single_and_matches_torch_on_representable_sums():
    # sums that are exactly representable in float32: rounding double -> bf16 equals torch's float32 -> bf16
    rng = np.random.default_rng(5)
    x = _bf16(rng.integers(-8, 9, size=(6, 128)).astype(np.float32))
    w = _bf16(rng.integers(-4, 5, size=(10, 128)).astype(np.float32))
    y, exact, _ = oracle.linear_bf16(x, w, None)
    ref = torch.from_numpy(exact.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(y, ref)
    # a tie between two bf16 values goes to the even one: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    one = _bf16(np.array([[1.0] + [0.0] * 127], np.float32))
    w2 = _bf16(np.array([[1.0] + [0.0] * 127], np.float32))
    y, _, _ = oracle.linear_bf16(one, w2, _bf16(np.array([2.0**-8], np.float32)))
    assert int(y[0, 0]) == 0x3F80
    y, _, _ = oracle.linear_bf16(one, w2, _bf16(np.array([3 * 2.0**-8], np.float32)))   # 1 + 3/256: tie -> 1 + 2/128 (even)
    assert int(y[0, 0]) == 0x3F82
