"""GPU parity of dp_wq_linear against the CPU oracle.

int8 codes, fp32 scales and int32 accumulators must be bit-exact; bf16 outputs within 1 bf16 ulp
(the kernels mirror the oracle's fp32 operation sequence, so 0 ulp is expected and asserted for
the vast majority)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import DevLayer, run_linear
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu
SEED = synth.BASE_SEED
# the tensor-core kernels that expand packed weights themselves (the default for packed layers is the
# unpack-first form, which runs the 8-bit kernel on an int8 copy: test_mma_path and
# test_mma_unpack_first cover it)
MMA_PACKED = B.DP_FLAG_FORCE_MMA | B.DP_FLAG_NO_UNPACK_FIRST


def _case(M, K, N, bits, layer=0, n_out=None, bias=True, full_range=False):
    x = synth.activations(SEED, layer, 0, M, K, 1.0, n_out=K // 100 if n_out is None else n_out)
    if full_range:  # every code incl. -2^(b-1)
        rng = np.random.default_rng(bits * 1000 + N)
        w = rng.integers(-(1 << (bits - 1)), 1 << (bits - 1), size=(N, K)).astype(np.int8)
        s_w = (np.abs(rng.standard_normal(N)) * 1e-3 + 1e-4).astype(np.float32)
    else:
        w, s_w = synth.weights(SEED, layer, N, K, bits)
    b = synth.bias(SEED, layer, N) if bias else None
    return x, w, s_w, b


def _check(out, x, w, s_w, b, bits, exact_y=True):
    y, q, s_a, acc = oracle.wq_linear(x, oracle.pack(w, bits), s_w, b, bits, taps=True)
    assert out["status"] == 0
    assert np.array_equal(out["s_a"].view(np.uint32), s_a.view(np.uint32)), "scales differ"
    assert np.array_equal(out["q"], q), "int8 codes differ"
    bad = np.argwhere(out["acc"] != acc)
    assert bad.size == 0, f"{len(bad)} accumulators differ, first at {bad[:5].tolist()}"
    d = bf16_ulp_dist(out["y"], y)
    assert d.max() <= 1, f"max bf16 distance {d.max()}"
    if exact_y:
        assert (d != 0).mean() < 1e-4


@pytest.mark.parametrize("bits", [3, 4, 8])
@pytest.mark.parametrize("M,K,N", [(1, 128, 32), (8, 1152, 96), (16, 1152, 6912), (21, 256, 48),
                                   (32, 4608, 64)])
def test_simt_path(bits, M, K, N):
    x, w, s_w, b = _case(M, K, N, bits, full_range=(N == 48))
    L = DevLayer(w, s_w, b, bits)
    _check(run_linear(L, x, flags=B.DP_FLAG_FORCE_SIMT), x, w, s_w, b, bits)


@pytest.mark.parametrize("bits", [8, 4, 3])
@pytest.mark.parametrize("M,K,N", [(128, 128, 64), (128, 256, 128), (256, 1152, 1152),
                                   (300, 1152, 384), (1000, 4608, 1152), (77, 384, 192),
                                   (2048, 1152, 4608)])
@pytest.mark.parametrize("unpack", [0, B.DP_FLAG_NO_UNPACK_FIRST], ids=["default", "in_gemm"])
def test_mma_path(bits, M, K, N, unpack):
    if bits == 8 and unpack:
        pytest.skip("8-bit weights have one form")
    x, w, s_w, b = _case(M, K, N, bits, full_range=(N in (64, 192)), bias=(N != 384))
    L = DevLayer(w, s_w, b, bits)
    _check(run_linear(L, x, flags=B.DP_FLAG_FORCE_MMA | unpack), x, w, s_w, b, bits)


@pytest.mark.parametrize("bits", [8, 4, 3])
@pytest.mark.parametrize("bn", [64, 128, 192, 256])
def test_mma_every_tile_width(bits, bn):
    """Each tile-width variant of the tensor-core kernel, several tiles per CTA is not needed for
    coverage of the variant itself: ragged M, two column tiles, K of three k-blocks."""
    M, K, N = 200, 384, 2 * bn
    x, w, s_w, b = _case(M, K, N, bits, full_range=True)
    L = DevLayer(w, s_w, b, bits)
    _check(run_linear(L, x, flags=MMA_PACKED | B.DP_FLAG_TILE_N(bn)), x, w, s_w, b, bits)


@pytest.mark.parametrize("bits", [8, 4, 3])
@pytest.mark.parametrize("bn", [128, 192, 256])
def test_mma_cta_pair_tiles(bits, bn):
    """The variant in which the two CTAs of a cluster share a 256-row tile (each holding half of
    the weight rows): ragged M (the second CTA's rows partly / wholly past M), two column tiles."""
    for M in (200, 100):
        K, N = 384, 2 * bn
        x, w, s_w, b = _case(M, K, N, bits, full_range=True)
        L = DevLayer(w, s_w, b, bits)
        _check(run_linear(L, x, flags=MMA_PACKED | B.DP_FLAG_CTA_PAIR | B.DP_FLAG_TILE_N(bn)),
               x, w, s_w, b, bits)


def test_mma_cta_pair_many_tiles():
    """More pair tiles than CTA pairs on the device: persistent loop, both accumulator buffers, ring
    wrap-around and the cross-CTA barriers over several rounds (M = 2100 -> 9 row tiles x 18)."""
    M, K, N = 2100, 256, 2304
    for bits in (8, 4, 3):
        x, w, s_w, b = _case(M, K, N, bits)
        L = DevLayer(w, s_w, b, bits)
        _check(run_linear(L, x, flags=MMA_PACKED | B.DP_FLAG_CTA_PAIR | B.DP_FLAG_TILE_N(128)),
               x, w, s_w, b, bits)


@pytest.mark.parametrize("bits", [8, 4, 3])
@pytest.mark.parametrize("N,K", [(384, 384), (512, 256), (768, 1152)])
def test_mma_weight_stationary(bits, N, K):
    """The CTA-pair kernel that keeps a strip of output channels resident for the whole K and streams
    only activation tiles: both strip widths (192, 256), short and full K, ragged M."""
    M = 600
    x, w, s_w, b = _case(M, K, N, bits, full_range=True)
    L = DevLayer(w, s_w, b, bits)
    _check(run_linear(L, x, flags=MMA_PACKED | B.DP_FLAG_WEIGHT_STATIONARY), x, w, s_w, b, bits)


def test_mma_weight_stationary_strip_changes():
    """More work items than CTA pairs, so pairs run several row tiles per strip and some runs cross
    a strip boundary (the resident strip is replaced while the pipeline is live)."""
    M, K, N = 2100, 1152, 2304
    for bits in (8, 4, 3):
        x, w, s_w, b = _case(M, K, N, bits)
        L = DevLayer(w, s_w, b, bits)
        _check(run_linear(L, x, flags=MMA_PACKED | B.DP_FLAG_WEIGHT_STATIONARY), x, w, s_w, b, bits)


AS = B.DP_FLAG_FORCE_MMA | B.DP_FLAG_ACT_STATIONARY


@pytest.mark.parametrize("bits", [8, 4, 3])
@pytest.mark.parametrize("bn", [64, 128, 192, 256])
@pytest.mark.parametrize("M,K", [(200, 384), (100, 1152), (600, 128)])
def test_mma_activation_stationary(bits, bn, M, K):
    """The CTA-pair kernel that keeps a 256-token strip of int8 codes resident for the whole K and
    streams only weight tiles: every sub-block width, short and full K (more and fewer k-blocks than
    ring stages), ragged M (the second CTA's tokens partly / wholly past M), several column
    sub-blocks per unit. Packed widths reach it through the unpack-first form."""
    N = 3 * bn
    x, w, s_w, b = _case(M, K, N, bits, full_range=True, bias=(bn != 128))
    L = DevLayer(w, s_w, b, bits)
    _check(run_linear(L, x, flags=AS | B.DP_FLAG_TILE_N(bn)), x, w, s_w, b, bits)


def test_mma_activation_stationary_several_units_and_strips_per_pair():
    """More units than CTA pairs: pairs run several units in a row, keep the resident strip across
    units of one strip and replace it while the weight ring is live when a run crosses strips; both
    accumulator buffers and the ring wrap around many times (M = 2100 -> 9 strips)."""
    for (M, K, N, bits, bn) in [(2100, 1152, 2304, 8, 64), (2100, 640, 2304, 4, 128), (5000, 1152, 1152, 3, 128),
                                (2100, 256, 4608, 8, 256)]:
        x, w, s_w, b = _case(M, K, N, bits)
        L = DevLayer(w, s_w, b, bits)
        _check(run_linear(L, x, flags=AS | B.DP_FLAG_TILE_N(bn)), x, w, s_w, b, bits)


@pytest.mark.parametrize("name,K,N", [("qkv", 1152, 3456), ("proj", 1152, 1152), ("fc1", 1152, 4608)])
def test_mma_activation_stationary_dit_shapes_default_sub_blocks(name, K, N):
    """The DiT-XL/2 shapes with K = 1152 at M = 2048, sub-block width chosen by the library (one unit
    per pair: 8 strips x 9 slices), 8-bit and packed weights."""
    for bits in (8, 4):
        x, w, s_w, b = _case(2048, K, N, bits, layer=3)
        L = DevLayer(w, s_w, b, bits)
        _check(run_linear(L, x, flags=AS), x, w, s_w, b, bits)


def test_mma_many_tiles_per_cta():
    """More tiles than SMs, so the persistent loop, both accumulator buffers and the stage ring
    wrap-around are exercised (M = 1300 -> 11 row tiles x 18 column tiles of 64)."""
    M, K, N = 1300, 256, 1152
    for bits in (8, 4, 3):
        x, w, s_w, b = _case(M, K, N, bits)
        L = DevLayer(w, s_w, b, bits)
        _check(run_linear(L, x, flags=MMA_PACKED | B.DP_FLAG_TILE_N(64)), x, w, s_w, b, bits)


@pytest.mark.parametrize("bits", [8, 4, 3])
def test_mma_one_hot_and_constant_inputs(bits):
    """One-hot tokens expose any permutation of k or n inside the tiles: acc[m,n] = 127*w[n,k_m]."""
    M, K, N = 128, 384, 128
    f = np.zeros((M, K), np.float32)
    for m in range(M):
        f[m, (m * 7) % K] = 1.0 if m % 2 == 0 else -2.0
    x = synth.f32_to_bf16_bits(f)
    rng = np.random.default_rng(bits)
    w = rng.integers(-(1 << (bits - 1)), 1 << (bits - 1), size=(N, K)).astype(np.int8)
    s_w = np.ones(N, np.float32)
    L = DevLayer(w, s_w, None, bits)
    out = run_linear(L, x, flags=MMA_PACKED)
    _check(out, x, w, s_w, None, bits)
    km = (np.arange(M) * 7) % K
    sign = np.where(np.arange(M) % 2 == 0, 127, -127)
    assert np.array_equal(out["acc"], sign[:, None] * w[:, km].T.astype(np.int32))
    xc = synth.f32_to_bf16_bits(np.full((M, K), 0.75, np.float32))
    _check(run_linear(L, xc, flags=MMA_PACKED), xc, w, s_w, None, bits)


@pytest.mark.parametrize("bits", [8, 4, 3])
def test_mma_extreme_accumulators(bits):
    """Saturated tokens against saturated weight rows at K = 4608: |acc| reaches 4608*127*2^(b-1)
    (7.5e7 at 8 bits, beyond 2^24), so the int32 -> fp32 step of the epilogue has to round; mixed
    with random rows and signs so every magnitude in between occurs too."""
    M, K, N = 128, 4608, 128
    rng = np.random.default_rng(bits + 100)
    f = rng.standard_normal((M, K)).astype(np.float32)
    f[0::4] = 3.0
    f[1::4] = -3.0
    f[2::4, ::2] = 1.0
    x = synth.f32_to_bf16_bits(f)
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    w = rng.integers(lo, hi + 1, size=(N, K)).astype(np.int8)
    w[0::4] = lo
    w[1::4] = hi
    w[2::4, : K // 2] = lo
    s_w = np.full(N, 2.0 ** -10, np.float32)
    L = DevLayer(w, s_w, None, bits)
    out = run_linear(L, x, flags=MMA_PACKED)
    assert np.abs(out["acc"]).max() == 4608 * 127 * (1 << (bits - 1))
    _check(out, x, w, s_w, None, bits)


@pytest.mark.parametrize("variant", [B.DP_FLAG_NO_CTA_PAIR, B.DP_FLAG_CTA_PAIR | B.DP_FLAG_NO_WEIGHT_STATIONARY,
                                     B.DP_FLAG_WEIGHT_STATIONARY, B.DP_FLAG_FORCE_SIMT],
                         ids=["single", "pair", "weight_stationary", "small_m_kernel"])
def test_padded_row_pitches_and_untouched_padding(variant):
    """x with ldx > K and y with ldy > N: the padding columns of y keep their contents, rows past M
    are not written, and the result equals the oracle's."""
    simt = variant == B.DP_FLAG_FORCE_SIMT
    M, K, N, bits = (20 if simt else 300), 256, 384, 4
    ldx, ldy, rows_alloc = K + 64, N + 40, M + 7
    x, w, s_w, b = _case(M, K, N, bits)
    L = DevLayer(w, s_w, b, bits)
    xp = np.full((M, ldx), 0x7FC0, np.uint16)  # NaN in the padding: must never be read into the result
    xp[:, :K] = x
    xd = torch.from_numpy(xp.view(np.int16).copy()).cuda().view(torch.bfloat16)
    y = torch.full((rows_alloc, ldy), 3.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, bits, variant), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flags = variant if simt else (variant | MMA_PACKED)
    B.dp_wq_linear(L.w, xd, ldx, None, M, y, ldy, ws, None, status, flags)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = y.view(torch.int16).cpu().numpy().view(np.uint16)
    ref = oracle.wq_linear(x, oracle.pack(w, bits), s_w, b, bits)
    assert bf16_ulp_dist(got[:M, :N], ref).max() <= 1
    assert np.all(got[:M, N:] == 0x4040) and np.all(got[M:, :] == 0x4040)  # bf16(3.0) untouched


def test_single_token_and_minimal_k_through_the_tensor_core_path():
    """M = 1 (one live row in a 128-row tile) and the smallest K (one k-block) on every variant."""
    for variant in (B.DP_FLAG_NO_CTA_PAIR, B.DP_FLAG_CTA_PAIR | B.DP_FLAG_NO_WEIGHT_STATIONARY,
                    B.DP_FLAG_WEIGHT_STATIONARY):
        for bits in (8, 3):
            x, w, s_w, b = _case(1, 128, 192, bits, full_range=True)
            L = DevLayer(w, s_w, b, bits)
            _check(run_linear(L, x, flags=MMA_PACKED | variant), x, w, s_w, b, bits, exact_y=False)


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("variant", [0, B.DP_FLAG_CTA_PAIR | B.DP_FLAG_NO_WEIGHT_STATIONARY,
                                     B.DP_FLAG_WEIGHT_STATIONARY])
@pytest.mark.parametrize("M,K,N", [(300, 1152, 384), (2048, 384, 768), (77, 128, 192)])
def test_mma_unpack_first(bits, variant, M, K, N):
    """Packed weights expanded once to int8 in the workspace (extra CTAs of the DAQ launch), then the
    8-bit kernel on the copy: every code value, ragged M, single-CTA / pair / weight-stationary."""
    x, w, s_w, b = _case(M, K, N, bits, full_range=True)
    L = DevLayer(w, s_w, b, bits)
    flags = B.DP_FLAG_FORCE_MMA | B.DP_FLAG_UNPACK_FIRST | variant
    in_gemm = (flags & ~B.DP_FLAG_UNPACK_FIRST) | B.DP_FLAG_NO_UNPACK_FIRST
    assert B.dp_wq_linear_workspace(M, N, K, bits, flags) - B.dp_wq_linear_workspace(M, N, K, bits, in_gemm) >= N * K
    _check(run_linear(L, x, flags=flags), x, w, s_w, b, bits)


@pytest.mark.parametrize("flags", [B.DP_FLAG_FORCE_SIMT, B.DP_FLAG_FORCE_MMA,
                                   B.DP_FLAG_FORCE_MMA | B.DP_FLAG_UNPACK_FIRST])
def test_prequantized_input(flags):
    M, K, N, bits = 130, 256, 128, 4
    x, w, s_w, b = _case(M, K, N, bits)
    q, s_a, _ = oracle.daq(x)
    L = DevLayer(w, s_w, b, bits)
    out = run_linear(L, x, flags=flags, prequant=(q, s_a), taps=False)
    y = oracle.wq_linear(x, oracle.pack(w, bits), s_w, b, bits)
    assert out["status"] == 0 and bf16_ulp_dist(out["y"], y).max() <= 1


def test_unpack_first_without_workspace_is_refused():
    """Quantized activations need no scratch, the int8 copy of the weights does: no launch without it."""
    M, K, N, bits = 130, 256, 128, 4
    x, w, s_w, b = _case(M, K, N, bits)
    q, s_a, _ = oracle.daq(x)
    L = DevLayer(w, s_w, b, bits)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(L.w, torch.from_numpy(q.copy()).cuda(), K, torch.from_numpy(s_a.copy()).cuda(), M, y, N, None,
                       None, status, B.DP_FLAG_FORCE_MMA | B.DP_FLAG_UNPACK_FIRST)
    assert e.value.status == B.DP_ERR_WORKSPACE


def test_default_dispatch_and_argument_errors():
    x, w, s_w, b = _case(16, 1152, 128, 8)
    L = DevLayer(w, s_w, b, 8)
    _check(run_linear(L, x), x, w, s_w, b, 8)            # small M -> streaming kernel
    x, w, s_w, b = _case(200, 1152, 128, 8)
    _check(run_linear(DevLayer(w, s_w, b, 8), x), x, w, s_w, b, 8)   # large M -> tensor cores
    y = torch.empty((16, 128), dtype=torch.bfloat16, device="cuda")
    xt = torch.empty((16, 1152), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    bad = B.make_weight(L.qweight, L.s_w, None, 128, 1152, 5)
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(bad, xt, 1152, None, 16, y, 128, ws)
    assert e.value.status == B.DP_ERR_BITS
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(L.w, xt, 1152, None, 16, y, 64, ws)
    assert e.value.status == B.DP_ERR_SHAPE
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(L.w, xt, 1152, None, 200, y, 128, None, flags=B.DP_FLAG_FORCE_MMA)
    assert e.value.status == B.DP_ERR_WORKSPACE
    B.dp_wq_linear(L.w, xt, 1152, None, 0, y, 128, ws)   # M = 0: no-op
