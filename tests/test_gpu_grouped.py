"""GPU parity of layers with group-wise weight scales (dp_weight.group_size > 0, optional zero-points)
against the oracle. Both sides run the same fp32 sequence (exact int32 sum per group, one fma per group
in order, one fma with the token scale and bias), so the bf16 outputs are expected equal; the bar is
1 bf16 ulp with almost all equal, as for the per-channel layers."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import to_dev_bf16, bf16_to_np
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu
SEED = synth.BASE_SEED + 32


class GroupedLayer:
    def __init__(self, N, K, bits, g, zeros, layer=0, bias=True, full_range=True):
        rng = np.random.default_rng(N * 7 + K + bits * 100 + g)
        half = 1 << (bits - 1)
        if full_range:
            self.w = rng.integers(-half, half, size=(N, K)).astype(np.int8)
        else:
            self.w, _ = synth.weights(SEED, layer, N, K, bits)
        self.s_w = (np.abs(rng.standard_normal((N, K // g))) * 1e-2 + 1e-4).astype(np.float32)
        self.z = rng.integers(0, 1 << bits, size=(N, K // g)).astype(np.uint8) if zeros else None
        self.b = synth.bias(SEED, layer, N) if bias else None
        self.bits, self.g, self.N, self.K = bits, g, N, K
        self.packed = oracle.pack(self.w, bits)
        dev = B.dp_pack_weights_host(self.w, bits)
        assert np.array_equal(dev.view(np.uint8).ravel(), self.packed.view(np.uint8).ravel())
        self.d_w = torch.from_numpy(dev.view(np.uint8).copy()).cuda()
        self.d_s = torch.from_numpy(self.s_w.copy()).cuda()
        self.d_z = None if self.z is None else torch.from_numpy(self.z.copy()).cuda()
        self.d_b = None if self.b is None else to_dev_bf16(self.b)
        self.dw = B.make_weight(self.d_w, self.d_s, self.d_b, N, K, bits, g, self.d_z)

    def ref(self, x):
        return oracle.wq_linear_grouped(x, self.packed, self.s_w, self.b, self.bits, self.g, self.z)


def _run(L, x):
    M = x.shape[0]
    y = torch.full((M, L.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.dp_wq_linear_workspace_grouped(M, L.dw), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dp_wq_linear(L.dw, to_dev_bf16(x), L.K, None, M, y, L.N, ws, None, st, 0)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return bf16_to_np(y)


def _check(got, ref):
    d = bf16_ulp_dist(got, ref)
    assert d.max() <= 1, int(d.max())
    assert (d != 0).mean() < 1e-4


@pytest.mark.parametrize("zeros", [False, True], ids=["symmetric", "zero_points"])
@pytest.mark.parametrize("bits", [8, 4, 3])
@pytest.mark.parametrize("g", [32, 64, 128, 192, 288])
def test_group_sizes_of_the_paper(g, bits, zeros):
    """Every group size the paper's plans use, at K = 1152 (all divide it: 36 .. 4 groups; 192 and 288
    straddle the 128-byte pipeline stages), ragged M, two column tiles, every code."""
    M, K, N = 200, 1152, 256
    L = GroupedLayer(N, K, bits, g, zeros, bias=(g != 64))
    x = synth.activations(SEED, 1, 0, M, K, 1.0, n_out=11)
    _check(_run(L, x), L.ref(x))


def test_grouped_small_m_long_k_and_many_tiles():
    """M = 16 (a grouped layer always takes the tensor-core path), K = 4608 with g = 128 (36 groups: the
    four tensor-memory buffers wrap nine times), and more tiles than SMs (persistent loop, buffers
    carried across tiles)."""
    for (M, K, N, bits, g, zeros) in [(16, 1152, 384, 4, 64, True), (300, 4608, 128, 8, 128, False),
                                      (1300, 256, 2304, 3, 32, True), (2048, 1152, 1152, 4, 128, False)]:
        L = GroupedLayer(N, K, bits, g, zeros, full_range=False)
        x = synth.activations(SEED, 2, 0, M, K, 1.0, n_out=max(1, K // 100))
        _check(_run(L, x), L.ref(x))


def test_plan_mixes_grouped_per_channel_and_16_bit_layers():
    from gpu_util import DevLayer
    K = 256
    Lg = GroupedLayer(128, K, 4, 64, True, layer=0)
    Lz = GroupedLayer(256, K, 8, 32, False, layer=1)
    w, s_w = synth.weights(SEED, 2, 192, K, 3)
    b = synth.bias(SEED, 2, 192)
    Lp = DevLayer(w, s_w, b, 3)
    plan = B.dp_plan_create([Lg.dw, Lp.w, Lz.dw], [300, 300, 24], B.DP_FLAG_GROUP_SMALL_M)
    try:
        kept = [1, 4]
        xs = [[synth.activations(SEED, l, t, M, K, synth.sigma_t(t, 10), n_out=2) for l, M in enumerate([300, 300, 24])]
              for t in kept]
        xd = [[to_dev_bf16(x) for x in row] for row in xs]
        ys = [[torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for M, N in [(300, 128), (300, 192), (24, 256)]]
              for _ in kept]
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dp_plan_run(plan, kept, 0, B.ptr_array([t.data_ptr() for row in xd for t in row]),
                      B.ptr_array([t.data_ptr() for row in ys for t in row]), ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        for i in range(len(kept)):
            _check(bf16_to_np(ys[i][0]), Lg.ref(xs[i][0]))
            assert bf16_ulp_dist(bf16_to_np(ys[i][1]), oracle.wq_linear(xs[i][1], oracle.pack(w, 3), s_w, b, 3)).max() <= 1
            _check(bf16_to_np(ys[i][2]), Lz.ref(xs[i][2]))
    finally:
        B.dp_plan_destroy(plan)


def test_grouped_argument_errors():
    L = GroupedLayer(128, 256, 4, 64, False)
    bad = B.make_weight(L.d_w, L.d_s, None, 128, 256, 4, 48)          # g % 32 != 0
    x = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(bad, x, 256, None, 8, y, 128, ws)
    assert e.value.status == B.DP_ERR_SHAPE
    with pytest.raises(B.DiffproError) as e:                          # workspace too small
        B.dp_wq_linear(L.dw, x, 256, None, 8, y, 128, ws[:256])
    assert e.value.status == B.DP_ERR_WORKSPACE
    zl = B.make_weight(L.d_w, L.d_s, None, 128, 256, 4, 0, L.d_s)     # zero-points without groups
    with pytest.raises(B.DiffproError) as e:
        B.dp_wq_linear(zl, x, 256, None, 8, y, 128, ws)
    assert e.value.status == B.DP_ERR_INVALID_ARG
