"""Pins for the oracle's packed-weight codec, integer GEMM, epilogue, whole layer and plan run."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import synth
from helpers import bf16_bits, bf16_ulp_dist, f32_frac, round_frac_to_f32

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bigint_pack(row, bits):
    """Independent restatement: the row's bit stream as one Python integer."""
    v = 0
    for k, w in enumerate(row):
        v |= (int(w) + (1 << (bits - 1))) << (bits * k)
    nw = (len(row) * bits + 31) // 32
    return [(v >> (32 * i)) & 0xFFFFFFFF for i in range(nw)]


def test_golden_words():
    for line in open(os.path.join(GOLD, "pack_words.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        lhs, rhs = line.split("->")
        toks = lhs.split()
        bits, w = int(toks[0]), np.array([[int(t) for t in toks[1:]]], np.int8)
        words = [int(t, 16) for t in rhs.split()]
        assert oracle.pack(w, bits)[0].tolist() == words
        assert np.array_equal(oracle.unpack(np.array([words], np.uint32), w.shape[1], bits), w)


@pytest.mark.parametrize("bits", [3, 4])
def test_every_code_at_every_position(bits):
    half = 1 << (bits - 1)
    K = 32
    for pos in range(K):
        for code in range(1 << bits):
            w = np.full((1, K), -half, np.int8)          # background code 0
            w[0, pos] = code - half
            p = oracle.pack(w, bits)
            assert p[0].tolist() == _bigint_pack(w[0], bits)
            assert np.array_equal(oracle.unpack(p, K, bits), w)
            w2 = np.full((1, K), half - 1, np.int8)      # background all-ones
            w2[0, pos] = code - half
            p2 = oracle.pack(w2, bits)
            assert p2[0].tolist() == _bigint_pack(w2[0], bits)
            assert np.array_equal(oracle.unpack(p2, K, bits), w2)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_roundtrip_random_both_directions(bits):
    rng = np.random.default_rng(bits)
    half = 1 << (bits - 1)
    w = rng.integers(-half, half, size=(7, 256)).astype(np.int8)
    p = oracle.pack(w, bits)
    assert np.array_equal(oracle.unpack(p, 256, bits), w)
    if bits != 8:
        words = rng.integers(0, 1 << 32, size=(5, 256 * bits // 32), dtype=np.uint64).astype(np.uint32)
        assert np.array_equal(oracle.pack(oracle.unpack(words, 256, bits), bits), words)
        for n in range(7):
            assert p[n].tolist() == _bigint_pack(w[n], bits)
    with pytest.raises(ValueError):
        if bits == 8:
            raise ValueError
        oracle.pack(np.full((1, 32), half, np.int8), bits)


def test_gemm_against_numpy_int64_and_structure():
    rng = np.random.default_rng(5)
    for (M, N, K) in [(3, 5, 128), (17, 33, 1152), (128, 64, 256)]:
        q = rng.integers(-127, 128, size=(M, K)).astype(np.int8)
        w = rng.integers(-128, 128, size=(N, K)).astype(np.int8)
        acc = oracle.gemm_i32(q, w)
        ref = q.astype(np.int64) @ w.astype(np.int64).T
        assert np.array_equal(acc.astype(np.int64), ref)
        assert np.abs(acc).max() <= K * 127 * 128
    # W = identity block: acc reproduces q (catches a transposed or mis-indexed operand)
    K = 128
    q = rng.integers(-127, 128, size=(9, K)).astype(np.int8)
    assert np.array_equal(oracle.gemm_i32(q, np.eye(K, dtype=np.int8)), q.astype(np.int32))
    # one-hot activation picks a weight column: acc[m, n] = 127 * w[n, k0]
    w = rng.integers(-8, 8, size=(40, K)).astype(np.int8)
    oh = np.zeros((1, K), np.int8)
    oh[0, 37] = 127
    assert np.array_equal(oracle.gemm_i32(oh, w)[0], 127 * w[:, 37].astype(np.int32))
    # extreme magnitudes at the largest K: no overflow
    q = np.full((1, 4608), -127, np.int8)
    w = np.full((1, 4608), -128, np.int8)
    assert oracle.gemm_i32(q, w)[0, 0] == 4608 * 127 * 128


def test_epilogue_exact_bound_and_bf16_rounding():
    rng = np.random.default_rng(9)
    M, N = 24, 40
    acc = rng.integers(-(7 * 10**7), 7 * 10**7, size=(M, N)).astype(np.int32)
    acc[0, :8] = [0, 1, -1, 2**24 + 1, -(2**24 + 3), 74907648, -74907648, 12345]
    s_a = (np.abs(rng.standard_normal(M)) * 0.05 + 1e-3).astype(np.float32)
    s_w = (np.abs(rng.standard_normal(N)) * 1e-3 + 1e-5).astype(np.float32)
    bias = synth.f32_to_bf16_bits((rng.standard_normal(N) * 0.5).astype(np.float32))
    y = oracle.epilogue(acc, s_a, s_w, bias)
    yf = synth.bf16_bits_to_f32(y)
    bf = synth.bf16_bits_to_f32(bias)
    for m in range(M):
        for n in range(N):
            prod = Fraction(int(acc[m, n])) * Fraction(float(s_a[m])) * Fraction(float(s_w[n]))
            exact = prod + Fraction(float(bf[n]))
            # fp32 pipeline error (int->fp32, one multiply, one fused rounding) + bf16 rounding
            tol = abs(prod) * Fraction(1, 2**22) + abs(exact) * Fraction(1, 2**24)
            tol += abs(exact) * Fraction(1, 2**8) + Fraction(1, 2**140)
            assert abs(Fraction(float(yf[m, n])) - exact) <= tol
    # same fp32 sequence evaluated with numpy float32/float64 + torch's bf16 rounding
    t = acc.astype(np.float32)
    sc = s_a[:, None] * s_w[None, :]
    y64 = t.astype(np.float64) * sc.astype(np.float64) + bf.astype(np.float64)[None, :]
    y32 = y64.astype(np.float32)  # double rounding can differ from a true fma only in rare ties
    ref = torch.from_numpy(y32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert bf16_ulp_dist(ref, y).max() <= 1
    assert (ref != y).mean() < 1e-3
    # bias = NULL means +0
    y0 = oracle.epilogue(acc, s_a, s_w, None)
    yz = oracle.epilogue(acc, s_a, s_w, np.zeros(N, np.uint16))
    assert np.array_equal(y0, yz)
    # s_w = 1, s_a = 1, small acc: y is the integer itself (exactly representable up to 256)
    a = np.arange(-256, 256, dtype=np.int32).reshape(1, -1)
    y1 = oracle.epilogue(a, np.ones(1, np.float32), np.ones(a.shape[1], np.float32), None)
    assert np.array_equal(synth.bf16_bits_to_f32(y1)[0], a[0].astype(np.float32))


def _bf16_rne_bits(v: np.float32) -> int:
    """bf16 bit pattern of a finite float32, round to nearest, ties to even, in exact rationals."""
    u = int(np.float32(v).view(np.uint32))
    lo = u & 0xFFFF0000                      # truncation toward zero (same sign)
    hi = lo + 0x10000                        # next bf16 away from zero
    f = lambda b: Fraction(float(np.uint32(b).view(np.float32)))
    x = Fraction(float(v))
    dl, dh = abs(x - f(lo)), abs(f(hi) - x)
    if dl < dh or (dl == dh and ((lo >> 16) & 1) == 0):
        return lo >> 16
    return hi >> 16


def _epilogue_sequences(acc: int, s_a, s_w, bias_f32):
    """Step 5's dequantisation of one accumulator in exact rationals, each fp32 operation rounded
    once to nearest-even: the defined sequence and two plausible wrong ones."""
    A, SA, SW, B = Fraction(acc), f32_frac(s_a), f32_frac(s_w), f32_frac(bias_f32)
    t = f32_frac(round_frac_to_f32(A))                         # int32 -> fp32
    sc = f32_frac(round_frac_to_f32(SA * SW))                  # s_a[m] * s_w[n]
    defined = round_frac_to_f32(t * sc + B)                    # one fused multiply-add
    other_assoc = round_frac_to_f32(f32_frac(round_frac_to_f32(t * SA)) * SW + B)   # (t*s_a)*s_w + bias
    unfused = round_frac_to_f32(f32_frac(round_frac_to_f32(t * sc)) + B)            # mul, then add
    return [_bf16_rne_bits(v) for v in (defined, other_assoc, unfused)]


def test_epilogue_exact_fp32_sequence():
    """orc_epilogue is exactly cvt(RN) -> s_a*s_w (RN) -> fma (RN) -> bf16 (RNE), evaluated here in
    exact rationals and compared for EQUALITY: random cases, |acc| > 2^24 (where the conversion
    rounds) and constructed cancellation cases acc*s_a*s_w ~ -bias, where the association
    (t*s_a)*s_w + bias and an unfused multiply-then-add land on other bf16 values. The test also
    checks that those two wrong sequences do differ from the oracle on its cases, so an oracle that
    computed either would fail here."""
    rng = np.random.default_rng(2511)
    cases = []
    for _ in range(300):                                        # random, full accumulator range
        cases.append((int(rng.integers(-(75 * 10**6), 75 * 10**6)),
                      np.float32(abs(rng.standard_normal()) * 0.05 + 1e-3),
                      np.float32(abs(rng.standard_normal()) * 1e-3 + 1e-5),
                      np.float32(rng.standard_normal() * 0.5)))
    for a in (2**24 + 1, -(2**24 + 3), 2**25 + 2, 2**26 - 1, 74907648, -74907648, 2**24 + 2, 33554433):
        cases.append((a, np.float32(0.0123), np.float32(3.3e-4), np.float32(-0.75)))
    for _ in range(400):                                        # cancellation: t*sc ~ -bias
        s_a = np.float32(abs(rng.standard_normal()) * 0.05 + 1e-3)
        s_w = np.float32(abs(rng.standard_normal()) * 1e-3 + 1e-5)
        b = np.float32(rng.standard_normal() * 2.0)
        b = np.float32(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.array([b], np.float32)))[0])
        a = int(round(-float(b) / (float(s_a) * float(s_w))))
        if abs(a) > 74907648 or a == 0:
            continue
        cases.append((a + int(rng.integers(-1, 2)), s_a, s_w, b))
    acc = np.array([[c[0] for c in cases]], np.int32).T.copy()          # [P, 1]: one row per case
    got = np.empty(len(cases), np.uint16)
    n_assoc = n_unfused = 0
    for i, (a, s_a, s_w, b) in enumerate(cases):
        bias_bits = synth.f32_to_bf16_bits(np.array([b], np.float32))
        bias_f32 = synth.bf16_bits_to_f32(bias_bits)[0]
        y = oracle.epilogue(acc[i:i + 1], np.array([s_a], np.float32), np.array([s_w], np.float32), bias_bits)
        got[i] = y[0, 0]
        want, assoc, unfused = _epilogue_sequences(a, s_a, s_w, bias_f32)
        assert int(got[i]) == want, (i, a, float(s_a), float(s_w), float(b))
        n_assoc += assoc != want
        n_unfused += unfused != want
    assert n_assoc >= 10 and n_unfused >= 10, (n_assoc, n_unfused)


def test_bf16_rounding_matches_torch_exhaustively_sampled():
    rng = np.random.default_rng(1)
    u = rng.integers(0, 1 << 32, size=200000, dtype=np.uint64).astype(np.uint32)
    f = u.view(np.float32)
    f = f[np.isfinite(f)]
    ties = (np.arange(1, 2000, dtype=np.uint32) << 16 | 0x8000).view(np.float32)  # exact halves
    f = np.concatenate([f, ties, -ties])
    mine = np.array([oracle.lib().orc_f32_to_bf16(float(v)) for v in f[:20000]], np.uint16)
    ref = torch.from_numpy(f[:20000].copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, ref)
    t = np.concatenate([ties, -ties])
    mine = np.array([oracle.lib().orc_f32_to_bf16(float(v)) for v in t], np.uint16)
    ref = torch.from_numpy(t.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, ref)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_whole_layer_composition_points_and_dequant_accuracy(bits):
    seed = synth.BASE_SEED + bits
    M, K, N = 48, 256, 80
    x = synth.activations(seed, 0, 0, M, K, 1.0, n_out=3)
    w, s_w = synth.weights(seed, 0, N, K, bits)
    b = synth.bias(seed, 0, N)
    pw = oracle.pack(w, bits)
    y, q, s_a, acc = oracle.wq_linear(x, pw, s_w, b, bits, taps=True)
    assert np.array_equal(oracle.wq_linear(x, pw, s_w, b, bits), y)
    assert np.array_equal(acc.astype(np.int64), q.astype(np.int64) @ w.astype(np.int64).T)
    rng = np.random.default_rng(0)
    pm, pn = rng.integers(0, M, 200), rng.integers(0, N, 200)
    pa, py = oracle.wq_linear_points(x, pw, s_w, b, bits, pm, pn)
    assert np.array_equal(pa, acc[pm, pn]) and np.array_equal(py, y[pm, pn])
    # the layer approximates the real-valued linear of the dequantized weights: the only error is
    # the activation rounding (<= s_a/2 per element) and the bf16 output rounding
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    wf = w.astype(np.float64) * s_w.astype(np.float64)[:, None]
    ref = xf @ wf.T + synth.bf16_bits_to_f32(b).astype(np.float64)[None, :]
    bound = (0.5 + 2.0**-15) * s_a.astype(np.float64)[:, None] * np.abs(wf).sum(axis=1)[None, :]
    got = synth.bf16_bits_to_f32(y).astype(np.float64)
    assert np.all(np.abs(got - ref) <= bound + np.abs(ref) * 2.0**-8 + 1e-6)


def test_plan_run_equals_independent_calls():
    seed = synth.BASE_SEED
    shapes = [(16, 128, 32, 8), (16, 128, 48, 4), (4, 256, 32, 3)]
    layers = []
    for l, (M, K, N, bits) in enumerate(shapes):
        w, s_w = synth.weights(seed, l, N, K, bits)
        layers.append(dict(M=M, N=N, K=K, bits=bits, qweight=oracle.pack(w, bits), s_w=s_w,
                           bias=synth.bias(seed, l, N) if l != 1 else None))
    kept = [2, 5, 9]
    xs = [[synth.activations(seed, l, t, L["M"], L["K"], synth.sigma_t(t, 10), n_out=2)
           for l, L in enumerate(layers)] for t in kept]
    ys = oracle.plan_run(layers, kept, xs)
    for i in range(len(kept)):
        for l, L in enumerate(layers):
            ref = oracle.wq_linear(xs[i][l], L["qweight"], L["s_w"], L["bias"], L["bits"])
            assert np.array_equal(ys[i][l], ref)
