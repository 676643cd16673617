"""dp_wq_linear_residual against the oracle: bit-for-bit (the epilogue is one fp32 sequence on both sides)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth

pytestmark = pytest.mark.gpu


def _run(M, K, N, bits, gate_rows, rpg, in_place, flags=0, seed=0):
    s = synth.BASE_SEED + 900 + seed
    x = synth.activations(s, 0, 0, M, K, 1.0, n_out=2)
    w, s_w = synth.weights(s, 0, N, K, bits)
    b = synth.bias(s, 0, N)
    res = synth.activations(s, 1, 0, M, N, 1.0, n_out=0)
    gate = None
    if gate_rows:
        rng = np.random.default_rng(s)
        gate = synth.f32_to_bf16_bits(rng.normal(0, 0.5, size=(-(-M // rpg), N)).astype(np.float32))
    pw = oracle.pack(w, bits)
    want = oracle.wq_linear_residual(x, pw, s_w, b, bits, res, gate, rpg)
    dev = "cuda:0"
    t = lambda a, dt: torch.from_numpy(a.view(dt) if dt is not None else a).to(dev)
    dx, dres = t(x, np.int16), t(res, np.int16)
    dgate = t(gate, np.int16) if gate is not None else None
    dpw, dsw, db = torch.from_numpy(pw).to(dev), t(s_w, None), t(b, np.int16)   # dp_weight holds raw pointers
    dw = B.make_weight(dpw, dsw, db, N, K, bits)
    fl = flags | B.DP_FLAG_FORCE_MMA | B.DP_FLAG_UNPACK_FIRST
    nws = B.dp_wq_linear_workspace(M, N, K, bits, fl)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    y = dres if in_place else torch.empty(M, N, dtype=torch.int16, device=dev)
    B.dp_wq_linear_residual(dw, dx, K, M, dres, N, dgate, rpg, y, N, ws, nws, status, flags)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = y.cpu().numpy().view(np.uint16)
    assert np.array_equal(got, want), (np.argwhere(got != want)[:5], M, K, N, bits)


@pytest.mark.parametrize("bits", [3, 4, 8])
@pytest.mark.parametrize("gated", [False, True])
def test_residual_small_and_ragged(bits, gated):
    _run(300, 256, 192, bits, gated, 77, False, seed=bits)


@pytest.mark.parametrize("tile", [64, 128, 192, 256])
@pytest.mark.parametrize("pair", [False, True])
def test_residual_every_tile_width(tile, pair):
    if pair and tile == 64:
        pytest.skip("pairs start at 128 columns")
    N = 768
    fl = ((tile // 64) << 8) | (B.DP_FLAG_CTA_PAIR if pair else B.DP_FLAG_NO_CTA_PAIR)
    _run(700, 384, N, 8, True, 256, False, flags=fl, seed=tile + pair)


def test_residual_in_place_dit_projection():
    # x <- x + gate * proj(attn): 2 samples of 1024 tokens (one DiT step's projection), written over x
    _run(2048, 1152, 1152, 4, True, 1024, True, seed=7)


def test_residual_argument_errors():
    dev = "cuda:0"
    M, K, N = 128, 128, 64
    z16 = torch.zeros(M, N, dtype=torch.int16, device=dev)
    x = torch.zeros(M, K, dtype=torch.int16, device=dev)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=dev)
    sw = torch.ones(N, device=dev)
    wt16 = torch.zeros(N, K, dtype=torch.int16, device=dev)
    w16 = B.dp_weight(N, K, 16, 0, wt16.data_ptr(), None, None)
    with pytest.raises(B.DiffproError):
        B.dp_wq_linear_residual(w16, x, K, M, z16, N, None, 1, z16, N, ws, ws.numel())
    w8 = B.make_weight(torch.zeros(N, K, dtype=torch.int8, device=dev), sw, None, N, K, 8)
    with pytest.raises(B.DiffproError):
        B.dp_wq_linear_residual(w8, x, K, M, z16, N - 8, None, 1, z16, N, ws, ws.numel())
    with pytest.raises(B.DiffproError):
        B.dp_wq_linear_residual(w8, x, K, M, z16, N, z16, 0, z16, N, ws, ws.numel())
    with pytest.raises(B.DiffproError):
        B.dp_wq_linear_residual(w8, x, K, M, z16, N, None, 1, z16, N, ws, ws.numel(), flags=B.DP_FLAG_FORCE_SIMT)
