"""Pins for the oracle's DAQ (Step 3, Eq. "daq"; b = 8, zero-point 0, tau = per-token absmax).

Each check is independent of the oracle's own code: exact rational arithmetic, closed forms, the
error bound of the equation, symmetries, and a library (torch CPU) cross-check of the absmax/scale.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import synth
from helpers import bf16_bits, f32_frac, round_frac_to_f32

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bf16(rng, shape, scale=1.0):
    return synth.f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def test_golden_half_to_even_ties():
    xs, qs = [], []
    for line in open(os.path.join(GOLD, "daq_ties.txt")):
        if line.strip() and not line.startswith("#"):
            a, b = line.split()
            xs.append(float(a))
            qs.append(int(b))
    x = bf16_bits(xs).reshape(1, -1)
    q, s_a, rowsum = oracle.daq(np.ascontiguousarray(x))
    assert s_a[0] == np.float32(1.0)
    assert q[0].tolist() == qs
    assert rowsum[0] == sum(qs)


def test_brute_force_exact_rational():
    rng = np.random.default_rng(7)
    for scale in (1.0, 37.5, 1e-3, 2.0**-90, 2.0**90):
        x = _rand_bf16(rng, (6, 24), scale)
        q, s_a, rowsum = oracle.daq(x)
        xf = synth.bf16_bits_to_f32(x)
        for m in range(x.shape[0]):
            fr = [Fraction(float(v)) for v in xf[m]]
            tau = max(abs(v) for v in fr)
            alpha = round_frac_to_f32(tau / 127)           # fl(tau / 127)
            inv = round_frac_to_f32(Fraction(127) / tau)   # fl(127 / tau)
            assert s_a[m] == alpha
            exp = [max(-127, min(127, round(v * Fraction(float(inv))))) for v in fr]  # half-even
            assert q[m].tolist() == exp
            assert rowsum[m] == sum(exp)


def test_error_bound_and_extremes():
    # |x - q*s_a| <= s_a * (1/2 + 2^-15): the real-number bound s_a/2 of the equation plus the
    # rounding of the two per-token divisions.
    x = synth.activations(synth.BASE_SEED, 0, 0, 64, 1152, 1.0, n_out=8)
    q, s_a, _ = oracle.daq(x)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    err = np.abs(xf - q.astype(np.float64) * s_a.astype(np.float64)[:, None])
    assert np.all(err <= s_a.astype(np.float64)[:, None] * (0.5 + 2.0**-15))
    # the absmax element maps to +-127 and nothing exceeds it
    am = np.abs(xf).argmax(axis=1)
    rows = np.arange(x.shape[0])
    assert np.all(np.abs(q[rows, am]) == 127)
    assert q.min() >= -127 and q.max() <= 127
    # scale is absmax/127 (torch CPU as an independent library evaluation)
    t = torch.from_numpy(xf.astype(np.float32))
    ref = (t.abs().amax(dim=-1) / 127.0).numpy()
    assert np.array_equal(ref.view(np.uint32), s_a.view(np.uint32))


def test_power_of_two_equivariance_and_sign_symmetry():
    rng = np.random.default_rng(3)
    x = _rand_bf16(rng, (16, 256))
    q, s_a, _ = oracle.daq(x)
    xf = synth.bf16_bits_to_f32(x)
    for j in (-20, -3, 5, 40):
        x2 = synth.f32_to_bf16_bits(xf * np.float32(2.0**j))
        q2, s2, _ = oracle.daq(x2)
        assert np.array_equal(q2, q)
        assert np.array_equal(s2, s_a * np.float32(2.0**j))
    qn, sn, rn = oracle.daq(x ^ np.uint16(0x8000))
    assert np.array_equal(qn, -q) and np.array_equal(sn, s_a)


def test_constant_zero_and_tiny_rows():
    c = np.full((1, 128), 3.25, np.float32)
    x = np.concatenate([bf16_bits(c), bf16_bits(-c), bf16_bits(np.zeros((1, 128))),
                        bf16_bits(np.full((1, 128), 2.0**-101)),
                        bf16_bits(np.full((1, 128), 2.0**-100))])
    q, s_a, rowsum = oracle.daq(x)
    assert np.all(q[0] == 127) and np.all(q[1] == -127)
    assert s_a[0] == np.float32(3.25) / np.float32(127)
    assert np.all(q[2] == 0) and s_a[2] == 0 and rowsum[2] == 0
    assert np.all(q[3] == 0) and s_a[3] == 0          # below the 2^-100 threshold: all-zero token
    assert np.all(q[4] == 127) and s_a[4] > 0         # at the threshold: quantized normally
    # a one-hot row: the single non-zero maps to +-127, the rest to 0
    oh = np.zeros((1, 128), np.float32)
    oh[0, 77] = -0.3125
    q, s_a, rowsum = oracle.daq(bf16_bits(oh))
    assert q[0, 77] == -127 and np.count_nonzero(q) == 1 and rowsum[0] == -127


def test_division_reading_disagreement_is_rare():
    """The reading 'multiply by fl(127/tau), round once' against 'RNE(fl(x / s_a))': they may
    differ by one step on a tiny fraction of elements; never by more."""
    x = synth.activations(synth.BASE_SEED, 1, 0, 256, 1152, 1.0, n_out=8)
    q, s_a, _ = oracle.daq(x)
    xf = synth.bf16_bits_to_f32(x)
    alt = np.rint(xf / s_a[:, None]).astype(np.int32)
    d = np.abs(alt - q.astype(np.int32))
    assert d.max() <= 1
    assert (d != 0).mean() < 1e-3


def test_strided_call_matches_contiguous():
    import ctypes as C
    rng = np.random.default_rng(11)
    M, K, ld = 5, 64, 96
    buf = _rand_bf16(rng, (M, ld))
    xc = np.ascontiguousarray(buf[:, :K])
    q0, s0, _ = oracle.daq(xc)
    q = np.zeros((M, ld), np.int8)
    s = np.zeros(M, np.float32)
    oracle.lib().orc_daq(buf.ctypes.data_as(C.c_void_p), C.c_int64(M), C.c_int64(K),
                         C.c_int64(ld), q.ctypes.data_as(C.c_void_p), C.c_int64(ld),
                         s.ctypes.data_as(C.c_void_p), None)
    assert np.array_equal(q[:, :K], q0) and np.array_equal(s, s0) and not q[:, K:].any()
