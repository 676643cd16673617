"""Pins for the oracle's DAQ with a percentile clip and a-bit codes (Step 3, Eq. "daq" with
tau = Percentile(|v|, p), p < 100; Step 6: activation bits per time bin).

Reading pinned here: nearest-rank percentile of one token's K magnitudes, handed over as its rank
from the top. Every check is independent of the oracle's code: exact rational arithmetic with
Python's own sort, numpy's inverted-CDF percentile, counting arguments, the equation's error bound,
symmetries, and the reduction to the (separately pinned) absmax DAQ.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_11446_b200 import synth
from helpers import round_frac_to_f32


def _rand_bf16(rng, shape, scale=1.0):
    return synth.f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def test_rank_one_eight_bits_is_the_absmax_daq():
    x = synth.activations(synth.BASE_SEED, 1, 0, 33, 1152, 1.0, n_out=11)
    (q, s_a, rowsum), (q0, s0, rowsum0) = oracle.daq_robust(x, 1, 8), oracle.daq(x)
    assert np.array_equal(q, q0) and np.array_equal(rowsum, rowsum0)
    assert np.array_equal(s_a.view(np.uint32), s0.view(np.uint32))


@pytest.mark.parametrize("p,K,rank", [("99.9", 1152, 2), ("99.9", 4608, 5), ("100", 1152, 1), ("99", 1152, 12),
                                      ("99.9", 128, 1), ("50", 128, 65), ("0.001", 128, 128)])
def test_rank_of_the_nearest_rank_percentile(p, K, rank):
    """ceil(p K / 100)-th smallest = (K - ceil(p K / 100) + 1)-th largest; numpy's inverted-CDF
    percentile is that same order statistic."""
    assert oracle.clip_rank(p, K) == rank
    rng = np.random.default_rng(K + rank)
    mag = np.abs(rng.standard_normal(K)).astype(np.float32)
    assert np.percentile(mag, float(p), method="inverted_cdf") == np.sort(mag)[::-1][rank - 1]


def test_brute_force_exact_rational():
    rng = np.random.default_rng(11)
    for scale in (1.0, 37.5, 1e-3, 2.0**-90, 2.0**90):
        for rank, bits in ((1, 8), (2, 8), (5, 8), (3, 4), (2, 2), (24, 6)):
            x = _rand_bf16(rng, (5, 24), scale)
            x[0, :6] = x[0, 6]  # repeated magnitudes: ranks count repeats
            q, s_a, rowsum = oracle.daq_robust(x, rank, bits)
            xf = synth.bf16_bits_to_f32(x)
            qmax = (1 << (bits - 1)) - 1
            for m in range(x.shape[0]):
                fr = [Fraction(float(v)) for v in xf[m]]
                tau = sorted((abs(v) for v in fr), reverse=True)[rank - 1]
                assert s_a[m] == round_frac_to_f32(tau / qmax)
                inv = Fraction(float(round_frac_to_f32(Fraction(qmax) / tau)))
                # the equation as written: clip to [-tau, tau] first, then round half to even ...
                clipped = [max(-tau, min(tau, v)) for v in fr]
                as_written = [round(v * inv) for v in clipped]
                # ... which never leaves the code range and equals round-then-clamp
                assert max(abs(c) for c in as_written) <= qmax
                exp = [max(-qmax, min(qmax, round(v * inv))) for v in fr]
                assert exp == as_written
                assert q[m].tolist() == exp
                assert rowsum[m] == sum(exp)


def test_clip_count_extremes_and_error_bound():
    K = 1152
    x = synth.activations(synth.BASE_SEED, 2, 7, 48, K, 1.7, n_out=11)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    for rank, bits in ((2, 8), (5, 8), (12, 6), (2, 4)):
        qmax = (1 << (bits - 1)) - 1
        q, s_a, _ = oracle.daq_robust(x, rank, bits)
        tau = np.sort(np.abs(xf), axis=1)[:, ::-1][:, rank - 1]
        # fewer than `rank` values lie strictly beyond the threshold, and all of them sit on an extreme code
        beyond = np.abs(xf) > tau[:, None]
        assert (beyond.sum(axis=1) <= rank - 1).all()
        assert (np.abs(q[beyond]) == qmax).all()
        assert (np.abs(q) <= qmax).all()
        # the threshold itself maps to +-qmax
        at = np.abs(xf) == tau[:, None]
        assert (np.abs(q[at]) == qmax).all()
        # inside the threshold the equation's bound holds: |x - q s_a| <= s_a (1/2 + qmax 2^-22)
        err = np.abs(xf - q.astype(np.float64) * s_a[:, None].astype(np.float64))
        bound = s_a.astype(np.float64) * (0.5 + qmax * 2.0**-22)
        assert (err[~beyond] <= np.broadcast_to(bound[:, None], err.shape)[~beyond]).all()


def test_symmetries_and_degenerate_rows():
    rng = np.random.default_rng(5)
    x = _rand_bf16(rng, (7, 256))
    q, s_a, _ = oracle.daq_robust(x, 3, 6)
    qn, sn, _ = oracle.daq_robust(x ^ np.uint16(0x8000), 3, 6)          # sign flip
    assert np.array_equal(qn, -q) and np.array_equal(sn, s_a)
    xs = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(x) * np.float32(2.0**9))  # power-of-two scaling
    q2, s2, _ = oracle.daq_robust(xs, 3, 6)
    assert np.array_equal(q2, q) and np.array_equal(s2, s_a * np.float32(2.0**9))
    # a row whose rank-th largest magnitude is zero quantizes to zero with scale zero
    z = np.zeros((1, 128), np.uint16)
    z[0, 5] = synth.f32_to_bf16_bits(np.array([3.0], np.float32))[0]
    q0, s0, r0 = oracle.daq_robust(z, 2, 8)
    assert not q0.any() and s0[0] == 0 and r0[0] == 0
    # constant rows land on the extreme code for every rank
    c = np.full((1, 128), synth.f32_to_bf16_bits(np.array([-0.75], np.float32))[0], np.uint16)
    for rank in (1, 64, 128):
        qc, _, _ = oracle.daq_robust(c, rank, 4)
        assert (qc == -7).all()
    with pytest.raises(ValueError):
        oracle.daq_robust(x, 0, 8)
    with pytest.raises(ValueError):
        oracle.daq_robust(x, 2, 9)
