"""Seeded synthetic inputs shaped like DiT-XL/2 linears (numpy side).

This module only GENERATES inputs (activations, integer weights, scales, biases, bit plans,
retained-timestep schedules). It holds none of the quantized-linear arithmetic and is the one piece
of code that both the CUDA tests and the CPU oracle tests consume. ``synth_cuda`` holds a CUDA
implementation of the same counter-based generators that is bit-identical to this one, for inputs
too large to make on the host.

Generator. Every tensor is a pure function of (seed, kind, layer, timestep, element index):
  stream key  = mix64 chain over (seed, kind, layer, t)
  element i   : two 64-bit hashes -> eight 16-bit uniforms -> their sum S (Irwin-Hall, n = 8)
                z = fp32(S - 262140) * fp32(1/53510.107)        (mean 0, variance 1, |z| < 4.9)
  activation  : bf16_rne( (z * sigma) * colscale[k] )           (fp32 multiplies, in this order)
  weight      : integer code w = clamp(rint(z / (max_k|z| / qmax)), -qmax, qmax), qmax = 2^(b-1)-1,
                scale s_w[n] = (max_k|z| / qmax) * 0.02         (symmetric round-to-nearest per
                output channel of a N(0, 0.02^2) matrix)
"""
from __future__ import annotations

import numpy as np

U64 = np.uint64
GOLDEN = U64(0x9E3779B97F4A7C15)
BASE_SEED = 0x25111446
IH_CENTER = 262140  # 8 * 65535 / 2
IH_INV_STD = np.float32(1.0 / 53510.107)

KIND_ACT, KIND_WEIGHT, KIND_BIAS, KIND_OUTLIER, KIND_PLAN, KIND_DRIFT = 1, 2, 3, 4, 5, 6

# DiT-XL/2: hidden 1152, MLP 4608, adaLN modulation 6 * 1152, 28 blocks.
HIDDEN, MLP, ADALN, BLOCKS = 1152, 4608, 6912, 28
# (name, K, N, rows-are-tokens)
BLOCK_LINEARS = (("qkv", HIDDEN, 3 * HIDDEN, True), ("proj", HIDDEN, HIDDEN, True),
                 ("fc1", HIDDEN, MLP, True), ("fc2", MLP, HIDDEN, True),
                 ("adaln", HIDDEN, ADALN, False))


def mix64(z):
    """splitmix64 finaliser on uint64 arrays (wrapping arithmetic)."""
    z = np.asarray(z, dtype=U64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> U64(30))) * U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> U64(27))) * U64(0x94D049BB133111EB)
        return z ^ (z >> U64(31))


def stream_key(seed: int, kind: int, layer: int = 0, t: int = 0) -> int:
    with np.errstate(over="ignore"):
        k = mix64(np.array([seed], U64) ^ (U64(kind) * GOLDEN))
        k = mix64(k + U64(layer) * GOLDEN + U64(1))
        k = mix64(k + U64(t) * GOLDEN + U64(2))
    return int(k[0])


def _sum16(h):
    m = U64(0xFFFF)
    return (h & m) + ((h >> U64(16)) & m) + ((h >> U64(32)) & m) + (h >> U64(48))


def std_normal(key: int, start: int, count: int) -> np.ndarray:
    """fp32 z for element indices start .. start+count-1 of stream `key`."""
    i = np.arange(start, start + count, dtype=U64)
    with np.errstate(over="ignore"):
        h0 = mix64(U64(key) + (U64(2) * i + U64(1)) * GOLDEN)
        h1 = mix64(U64(key) + (U64(2) * i + U64(2)) * GOLDEN)
    s = (_sum16(h0) + _sum16(h1)).astype(np.int64) - IH_CENTER
    return s.astype(np.float32) * IH_INV_STD


def f32_to_bf16_bits(f: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even of finite float32 to bf16 bit patterns (uint16)."""
    u = np.ascontiguousarray(f, np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(
        np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def outlier_colscale(seed: int, layer: int, t: int, K: int, n_out: int, factor: float = 20.0):
    """fp32 [K] column multipliers: `factor` on n_out seeded channels, 1 elsewhere."""
    key = stream_key(seed, KIND_OUTLIER, layer, t)
    with np.errstate(over="ignore"):
        h = mix64(U64(key) + (np.arange(K, dtype=U64) + U64(1)) * GOLDEN)
    cols = np.argsort(h, kind="stable")[:n_out]
    cs = np.ones(K, np.float32)
    cs[cols] = np.float32(factor)
    return cs


def activations(seed: int, layer: int, t: int, M: int, K: int, sigma: float = 1.0,
                n_out: int = 0, factor: float = 20.0, rows=None) -> np.ndarray:
    """bf16 bits [M,K] (or the selected `rows`): N(0, sigma^2) with n_out outlier channels."""
    key = stream_key(seed, KIND_ACT, layer, t)
    cs = outlier_colscale(seed, layer, t, K, n_out, factor)
    if rows is None:
        z = std_normal(key, 0, M * K).reshape(M, K)
    else:
        z = np.stack([std_normal(key, int(r) * K, K) for r in rows])
    return f32_to_bf16_bits((z * np.float32(sigma)) * cs[None, :])


def gelu_activations(seed: int, layer: int, t: int, M: int, K: int) -> np.ndarray:
    """bf16 bits of GELU(z), z ~ N(0,1): the skewed, non-negative-heavy input an MLP's second
    linear sees. Host only (erf in double)."""
    from math import sqrt
    try:
        from scipy.special import erf
    except Exception:  # pragma: no cover
        erf = np.vectorize(__import__("math").erf)
    z = std_normal(stream_key(seed, KIND_ACT, layer, t), 0, M * K).astype(np.float64)
    g = 0.5 * z * (1.0 + erf(z / sqrt(2.0)))
    return f32_to_bf16_bits(g.astype(np.float32)).reshape(M, K)


def weights(seed: int, layer: int, N: int, K: int, bits: int):
    """(w int8 [N,K] codes in [-qmax, qmax], s_w fp32 [N])."""
    key = stream_key(seed, KIND_WEIGHT, layer, 0)
    qmax = np.float32((1 << (bits - 1)) - 1)
    w = np.empty((N, K), np.int8)
    s_w = np.empty(N, np.float32)
    step = max(1, (1 << 22) // K)
    for n0 in range(0, N, step):
        n1 = min(N, n0 + step)
        z = std_normal(key, n0 * K, (n1 - n0) * K).reshape(n1 - n0, K)
        amax = np.abs(z).max(axis=1)
        s = np.where(amax > 0, amax / qmax, np.float32(1.0)).astype(np.float32)
        w[n0:n1] = np.clip(np.rint(z / s[:, None]), -qmax, qmax).astype(np.int8)
        s_w[n0:n1] = s * np.float32(0.02)
    return w, s_w


def bias(seed: int, layer: int, N: int, std: float = 0.01) -> np.ndarray:
    """bf16 bits [N] ~ N(0, std^2)."""
    z = std_normal(stream_key(seed, KIND_BIAS, layer, 0), 0, N)
    return f32_to_bf16_bits(z * np.float32(std))


def bit_plan(seed: int, n_layers: int, choices=(3, 4, 8)) -> list[int]:
    """Per-layer weight bit-widths drawn uniformly from `choices`."""
    key = stream_key(seed, KIND_PLAN)
    with np.errstate(over="ignore"):
        h = mix64(U64(key) + (np.arange(n_layers, dtype=U64) + U64(1)) * GOLDEN)
    return [choices[int(v % U64(len(choices)))] for v in h]


def kept_timesteps(seed: int, T: int = 50, keep: int = 25, rho: float = 0.2) -> list[int]:
    """A retained-timestep list shaped like Step 4's rule: the protected tail {t : t/T >= 1-rho}
    plus the highest-drift steps of the rest, with a stand-in drift exp(-t/10)*(1+jitter) (the
    paper's measured drift needs its models). Ascending order."""
    key = stream_key(seed, KIND_DRIFT)
    with np.errstate(over="ignore"):
        h = mix64(U64(key) + (np.arange(T, dtype=U64) + U64(1)) * GOLDEN)
    jitter = (h >> U64(40)).astype(np.float64) / float(1 << 24) * 0.1
    drift = np.exp(-np.arange(T) / 10.0) * (1.0 + jitter)
    tail = [t for t in range(T) if t / T >= 1.0 - rho]
    rest = [t for t in range(T) if t not in tail]
    top = sorted(rest, key=lambda t: -drift[t])[:max(0, keep - len(tail))]
    return sorted(tail + top)


def dit_layers(batch: int, tokens: int, blocks: int = BLOCKS):
    """[(name, M, K, N)] for `blocks` DiT-XL/2 blocks: token linears at M = batch*tokens, the adaLN
    modulation linear at M = batch."""
    out = []
    for b in range(blocks):
        for name, K, N, tok in BLOCK_LINEARS:
            out.append((f"b{b}.{name}", batch * tokens if tok else batch, K, N))
    return out


def sigma_t(t: int, T: int) -> float:
    """Activation std drifting with the timestep: 0.5 + 2 t / T."""
    return 0.5 + 2.0 * t / T
