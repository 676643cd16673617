"""Pins for the oracle's LayerNorm + adaLN modulation + DAQ (the operator in front of a DiT block's qkv
and fc1 linears taken into their activation quantization)."""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import synth
from helpers import f32_frac, round_frac_to_f32

EPS = 1e-6


def _inputs(M, K, seed, rows_per_sample):
    s = synth.BASE_SEED + 300 + seed
    x = synth.activations(s, 0, 0, M, K, 1.0, n_out=max(1, K // 100))
    rng = np.random.default_rng(s)
    S = -(-M // rows_per_sample)
    shift = synth.f32_to_bf16_bits(rng.normal(0, 0.3, (S, K)).astype(np.float32))
    scale = synth.f32_to_bf16_bits(rng.normal(0, 0.3, (S, K)).astype(np.float32))
    return x, shift, scale


def _sqrt_to_double(fr: Fraction) -> float:
    """Correctly rounded double of sqrt(fr), from an integer square root carried to 2^-200."""
    n = fr.numerator << 400
    r = math.isqrt(n // fr.denominator)          # floor(sqrt(fr) * 2^200)
    return float(Fraction(r, 1 << 200))


def test_fp32_sequence_in_exact_arithmetic():
    """Every rounding step written out with exact rationals: sums exact, mean and variance rounded to
    double, sqrt and reciprocal to double, both to fp32; then fp32 subtract, multiply, 1 + scale, fma.
    A population/sample variance mix-up, eps outside the root, a fused (x - mean) * rstd or scale applied
    without the 1 all land on other bits."""
    M, K, rps = 5, 48, 2
    x, shift, scale = _inputs(M, K, 1, rps)
    _, _, h = oracle.ln_modulate_daq(x, shift, scale, rps, EPS, tap=True)
    xf, shf, scf = (synth.bf16_bits_to_f32(t) for t in (x, shift, scale))
    eps_d = Fraction(float(np.float32(EPS)))
    for m in range(M):
        xs = [f32_frac(v) for v in xf[m]]
        mean_d = Fraction(float(sum(xs) / K))
        ex2_d = Fraction(float(sum(v * v for v in xs) / K))
        var_d = Fraction(float(ex2_d - Fraction(float(mean_d * mean_d))))
        sd = Fraction(_sqrt_to_double(Fraction(float(var_d + eps_d))))
        rstd32 = f32_frac(round_frac_to_f32(Fraction(float(1 / sd))))
        mean32 = f32_frac(round_frac_to_f32(mean_d))
        for k in range(K):
            d = f32_frac(round_frac_to_f32(xs[k] - mean32))
            n = f32_frac(round_frac_to_f32(d * rstd32))
            g = f32_frac(round_frac_to_f32(1 + f32_frac(scf[m // rps, k])))
            want = round_frac_to_f32(n * g + f32_frac(shf[m // rps, k]))
            assert h[m, k].view(np.uint32) == want.view(np.uint32), (m, k)


def test_against_library_layer_norm_in_double():
    M, K, rps = 64, 1152, 16
    x, shift, scale = _inputs(M, K, 2, rps)
    _, _, h = oracle.ln_modulate_daq(x, shift, scale, rps, EPS, tap=True)
    xd = torch.from_numpy(synth.bf16_bits_to_f32(x).astype(np.float64))
    ref = torch.nn.functional.layer_norm(xd, (K,), eps=float(np.float32(EPS)))
    sc = torch.from_numpy(synth.bf16_bits_to_f32(scale).astype(np.float64)).repeat_interleave(rps, 0)[:M]
    sh = torch.from_numpy(synth.bf16_bits_to_f32(shift).astype(np.float64)).repeat_interleave(rps, 0)[:M]
    ref = (ref * (1 + sc) + sh).numpy()
    # four fp32 roundings on values of magnitude <= |n| (1 + |scale|) + |shift|
    tol = 2.0**-22 * (np.abs(ref) + np.abs(sh.numpy()) + 1.0)
    assert np.all(np.abs(h - ref) <= tol)
    # without modulation: zero mean, unit variance per token (up to fp32)
    _, _, n = oracle.ln_modulate_daq(x, None, None, 1, EPS, tap=True)
    assert np.all(np.abs(n.astype(np.float64).mean(1)) < 1e-6)
    assert np.all(np.abs((n.astype(np.float64) ** 2).mean(1) - 1.0) < 1e-4)


def test_quantization_stage_is_eq_daq_on_the_fp32_activations():
    M, K, rps = 40, 384, 8
    x, shift, scale = _inputs(M, K, 3, rps)
    q, s_a, h = oracle.ln_modulate_daq(x, shift, scale, rps, EPS, tap=True)
    a = np.abs(h).max(1)
    assert np.array_equal(s_a.view(np.uint32), (a / np.float32(127.0)).astype(np.float32).view(np.uint32))
    am = np.abs(h).argmax(1)
    assert np.all(np.abs(q[np.arange(M), am]) == 127) and np.abs(q).max() <= 127
    err = np.abs(h.astype(np.float64) - q.astype(np.float64) * s_a[:, None].astype(np.float64))
    assert np.all(err <= s_a[:, None].astype(np.float64) * (0.5 + 2.0**-20))
    # brute force in exact rationals on a few tokens: one rounding of the exact product with fl(127 / a)
    for m in (0, 17, 39):
        inv = f32_frac(np.float32(127.0) / a[m])
        for k in range(0, K, 37):
            e = f32_frac(h[m, k]) * inv
            r = math.floor(e + Fraction(1, 2))
            if e + Fraction(1, 2) == r and r % 2:   # tie: to even
                r -= 1
            assert int(q[m, k]) == max(-127, min(127, r))


def test_special_cases():
    M, K = 6, 128
    x, shift, scale = _inputs(M, K, 4, 3)
    zeros = np.zeros_like(shift)
    a = oracle.ln_modulate_daq(x, zeros, zeros, 3, EPS)
    b = oracle.ln_modulate_daq(x, None, None, 1, EPS)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])      # 1 + 0 and + 0 change nothing
    const = np.full((M, K), synth.f32_to_bf16_bits(np.array([1.5], np.float32))[0], np.uint16)
    q, s_a, h = oracle.ln_modulate_daq(const, shift, scale, 3, EPS, tap=True)
    assert np.array_equal(h, synth.bf16_bits_to_f32(shift).repeat(3, 0)[:M])   # zero variance: only the shift is left
    q0, s0 = oracle.ln_modulate_daq(const, None, None, 1, EPS)
    assert not q0.any() and not s0.any()                                    # and without it an all-zero token
    # a power-of-two rescaling of the token leaves the normalized values where eps does not matter
    big = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(x) * np.float32(64.0))
    _, _, n1 = oracle.ln_modulate_daq(x, None, None, 1, 0.0, tap=True)
    _, _, n2 = oracle.ln_modulate_daq(big, None, None, 1, 0.0, tap=True)
    assert np.array_equal(n1, n2)
