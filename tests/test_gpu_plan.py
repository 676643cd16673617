"""GPU parity of dp_plan_run (Algorithm 2, Phase B over the linears) against the oracle."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import DevLayer, to_dev_bf16, bf16_to_np
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu
SEED = synth.BASE_SEED + 4


def _mini_plan(tokens=256, batch=2, blocks=2):
    """A scaled-down DiT stack: same five linears per block, mixed {3,4,8} plan."""
    table = synth.dit_layers(batch, tokens, blocks)
    bits = synth.bit_plan(SEED, len(table))
    layers, dev = [], []
    for l, (name, M, K, N) in enumerate(table):
        w, s_w = synth.weights(SEED, l, N, K, bits[l])
        b = synth.bias(SEED, l, N)
        dev.append(DevLayer(w, s_w, b, bits[l]))
        layers.append(dict(M=M, N=N, K=K, bits=bits[l], qweight=oracle.pack(w, bits[l]), s_w=s_w, bias=b))
    return table, layers, dev


def test_plan_run_matches_oracle_every_step_and_layer():
    table, layers, dev = _mini_plan()
    T = 10
    kept = synth.kept_timesteps(SEED, T, 4, 0.2)
    nL, nS = len(layers), len(kept)
    xs = [[synth.activations(SEED, l, t, L["M"], L["K"], synth.sigma_t(t, T), n_out=max(1, L["K"] // 100))
           for l, L in enumerate(layers)] for t in kept]
    ref = oracle.plan_run(layers, kept, xs)
    plan = B.dp_plan_create([d.w for d in dev], [L["M"] for L in layers])
    try:
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        xd = [[to_dev_bf16(xs[i][l]) for l in range(nL)] for i in range(nS)]
        yd = [[torch.full((L["M"], L["N"]), float("nan"), dtype=torch.bfloat16, device="cuda")
               for L in layers] for _ in range(nS)]
        xp = B.ptr_array([xd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        yp = B.ptr_array([yd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        B.dp_plan_run(plan, kept, 0, xp, yp, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for i in range(nS):
            for l in range(nL):
                d = bf16_ulp_dist(bf16_to_np(yd[i][l]), ref[i][l])
                assert d.max() <= 1, (i, l, table[l], int(d.max()))
        # resume: with start_index = 1 the last kept step (visited first) is skipped
        for i in range(nS):
            for l in range(nL):
                yd[i][l].fill_(float("nan"))
        B.dp_plan_run(plan, kept, 1, xp, yp, ws, status)
        torch.cuda.synchronize()
        assert torch.isnan(yd[nS - 1][0].float()).all()
        assert bf16_ulp_dist(bf16_to_np(yd[0][1]), ref[0][1]).max() <= 1
        # SAME_Y: every step overwrites one output set; the last write is kept[0]'s (reverse order)
        ys = [torch.empty((L["M"], L["N"]), dtype=torch.bfloat16, device="cuda") for L in layers]
        B.dp_plan_run(plan, kept, 0, xp, B.ptr_array([t.data_ptr() for t in ys]), ws, status,
                      flags=B.DP_PLAN_SAME_Y)
        torch.cuda.synchronize()
        for l in range(nL):
            assert bf16_ulp_dist(bf16_to_np(ys[l]), ref[0][l]).max() <= 1
        # the same run captured in a CUDA graph and replayed
        g = torch.cuda.CUDAGraph()
        for t in ys:
            t.zero_()
        side = torch.cuda.Stream()
        with torch.cuda.graph(g, stream=side):
            B.dp_plan_run(plan, kept, 0, xp, B.ptr_array([t.data_ptr() for t in ys]), ws, status,
                          flags=B.DP_PLAN_SAME_Y)
        g.replay()
        torch.cuda.synchronize()
        for l in range(nL):
            assert bf16_ulp_dist(bf16_to_np(ys[l]), ref[0][l]).max() <= 1
        assert int(status.item()) == 0
    finally:
        B.dp_plan_destroy(plan)


@pytest.mark.parametrize("extra", [B.DP_FLAG_FUSED_DAQ, 0], ids=["daq_in_gemm", "daq_kernel"])
def test_plan_autotuned_and_grouped_matches_oracle(extra):
    """Plan created with the on-device autotuner and with the small-M layers (adaLN) of a step
    grouped into one launch, with DAQ inside the GEMM kernels or in its own kernel (default): every
    output of every step still equals the oracle's."""
    table, layers, dev = _mini_plan(tokens=256, batch=3, blocks=3)
    T = 6
    kept = [1, 4, 5]
    nL, nS = len(layers), len(kept)
    xs = [[synth.activations(SEED, l, t, L["M"], L["K"], synth.sigma_t(t, T), n_out=max(1, L["K"] // 100))
           for l, L in enumerate(layers)] for t in kept]
    ref = oracle.plan_run(layers, kept, xs)
    plan = B.dp_plan_create([d.w for d in dev], [L["M"] for L in layers],
                            B.DP_FLAG_AUTOTUNE | B.DP_FLAG_GROUP_SMALL_M | extra)
    try:
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        xd = [[to_dev_bf16(xs[i][l]) for l in range(nL)] for i in range(nS)]
        yd = [[torch.full((L["M"], L["N"]), float("nan"), dtype=torch.bfloat16, device="cuda")
               for L in layers] for _ in range(nS)]
        xp = B.ptr_array([xd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        yp = B.ptr_array([yd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        B.dp_plan_run(plan, kept, 0, xp, yp, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for i in range(nS):
            for l in range(nL):
                d = bf16_ulp_dist(bf16_to_np(yd[i][l]), ref[i][l])
                assert d.max() <= 1, (i, l, table[l], int(d.max()))
    finally:
        B.dp_plan_destroy(plan)


def test_plan_with_variants_set_per_layer_matches_oracle():
    """dp_plan_set_layer_flags: every tensor-core layer switched to another variant after creation
    (unpack-first for the packed ones, CTA pairs / forced widths for the rest), workspace asked again,
    every output still the oracle's; small-M layers and nonsense flags are refused."""
    table, layers, dev = _mini_plan(tokens=256, batch=2, blocks=2)
    T, kept = 6, [2, 5]
    nL, nS = len(layers), len(kept)
    xs = [[synth.activations(SEED, l, t, L["M"], L["K"], synth.sigma_t(t, T), n_out=max(1, L["K"] // 100))
           for l, L in enumerate(layers)] for t in kept]
    ref = oracle.plan_run(layers, kept, xs)
    plan = B.dp_plan_create([d.w for d in dev], [L["M"] for L in layers],
                            B.DP_FLAG_GROUP_SMALL_M | B.DP_FLAG_NO_UNPACK_FIRST)
    try:
        before = B.dp_plan_workspace(plan)
        choices = [B.DP_FLAG_UNPACK_FIRST | B.DP_FLAG_TILE_N(128) | B.DP_FLAG_NO_CTA_PAIR,
                   B.DP_FLAG_CTA_PAIR | B.DP_FLAG_NO_WEIGHT_STATIONARY | B.DP_FLAG_UNPACK_FIRST,
                   B.DP_FLAG_TILE_N(64) | B.DP_FLAG_NO_CTA_PAIR | B.DP_FLAG_NO_UNPACK_FIRST]
        n_set = 0
        for l, L in enumerate(layers):
            if B.dp_plan_layer_variant(plan, l)["small_m"]:
                with pytest.raises(B.DiffproError):
                    B.dp_plan_set_layer_flags(plan, l, B.DP_FLAG_UNPACK_FIRST)
                continue
            B.dp_plan_set_layer_flags(plan, l, choices[n_set % 3])
            v = B.dp_plan_layer_variant(plan, l)
            assert v["unpack_first"] == (1 if (choices[n_set % 3] & B.DP_FLAG_UNPACK_FIRST) and L["bits"] < 8 else 0)
            if choices[n_set % 3] & B.DP_FLAG_TILE_N_MASK:
                assert v["tile_n"] == ((choices[n_set % 3] & B.DP_FLAG_TILE_N_MASK) >> 8) * 64
            n_set += 1
        with pytest.raises(B.DiffproError):
            B.dp_plan_set_layer_flags(plan, 0, B.DP_FLAG_FORCE_MMA)
        assert n_set >= 8 and B.dp_plan_workspace(plan) > before
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        xd = [[to_dev_bf16(xs[i][l]) for l in range(nL)] for i in range(nS)]
        yd = [[torch.full((L["M"], L["N"]), float("nan"), dtype=torch.bfloat16, device="cuda")
               for L in layers] for _ in range(nS)]
        xp = B.ptr_array([xd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        yp = B.ptr_array([yd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        B.dp_plan_run(plan, kept, 0, xp, yp, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for i in range(nS):
            for l in range(nL):
                d = bf16_ulp_dist(bf16_to_np(yd[i][l]), ref[i][l])
                assert d.max() <= 1, (i, l, table[l], int(d.max()))
    finally:
        B.dp_plan_destroy(plan)


@pytest.mark.parametrize("flags", [B.DP_FLAG_GROUP_SMALL_M, B.DP_FLAG_NO_UNPACK_FIRST | B.DP_FLAG_FUSED_DAQ],
                         ids=["grouped", "in_gemm_fused"])
def test_plan_with_daq_policy_matches_oracle_composition(flags):
    """dp_plan_set_daq: percentile clip (p = 99.9) and activation bits per time bin (8 / 6 / 4 for
    the thirds of 12 timesteps) on every layer, whatever variants the plan was created with; the
    oracle composes its pinned pieces step by step. Setting the policy back restores the plain rule."""
    table, layers, dev = _mini_plan(tokens=256, batch=2, blocks=1)
    T, kept, by_bin = 12, [1, 5, 6, 11], [8, 6, 4]
    nL, nS = len(layers), len(kept)
    xs = [[synth.activations(SEED, l, t, L["M"], L["K"], synth.sigma_t(t, T), n_out=max(1, L["K"] // 100))
           for l, L in enumerate(layers)] for t in kept]

    def compose(p, bins):
        out = []
        for i, t in enumerate(kept):
            bits = bins[min(2, 3 * t // T)]
            row = []
            for l, L in enumerate(layers):
                q, s_a, _ = oracle.daq_robust(xs[i][l], oracle.clip_rank(p, L["K"]), bits)
                w = oracle.unpack(L["qweight"], L["K"], L["bits"])
                row.append(oracle.epilogue(oracle.gemm_i32(q, w), s_a, L["s_w"], L["bias"]))
            out.append(row)
        return out

    plan = B.dp_plan_create([d.w for d in dev], [L["M"] for L in layers], flags)
    try:
        xd = [[to_dev_bf16(xs[i][l]) for l in range(nL)] for i in range(nS)]
        xp = B.ptr_array([xd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for p_e3, p, bins in ((99900, "99.9", by_bin), (100000, "100", [8, 8, 8])):
            B.dp_plan_set_daq(plan, p_e3, T, bins)
            ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
            yd = [[torch.full((L["M"], L["N"]), float("nan"), dtype=torch.bfloat16, device="cuda")
                   for L in layers] for _ in range(nS)]
            yp = B.ptr_array([yd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
            B.dp_plan_run(plan, kept, 0, xp, yp, ws, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            ref = compose(p, bins)
            for i in range(nS):
                for l in range(nL):
                    d = bf16_ulp_dist(bf16_to_np(yd[i][l]), ref[i][l])
                    assert d.max() <= 1, (p, i, l, table[l], int(d.max()))
        with pytest.raises(B.DiffproError):
            B.dp_plan_set_daq(plan, 99900, T, [8, 9, 4])
        with pytest.raises(B.DiffproError):
            B.dp_plan_set_daq(plan, 90000, T, by_bin)  # K = 1152 would need rank 116
    finally:
        B.dp_plan_destroy(plan)


def test_daq_policy_on_grouped_small_m_layers_with_long_rows():
    """Small-M layers of equal shape are grouped; under a DAQ policy a group with K = 4608 cannot use
    the grouped quantization kernel (rows up to 1280) and falls back to layer-by-layer launches, a
    group with K = 1152 keeps its shared launch: both must equal the oracle's composition."""
    shapes = [(8, 4608, 256, 4), (8, 4608, 256, 8), (8, 1152, 96, 3), (8, 1152, 96, 4), (16, 1152, 96, 8)]
    layers, dev = [], []
    for l, (M, K, N, bits) in enumerate(shapes):
        w, s_w = synth.weights(SEED, 40 + l, N, K, bits)
        b = synth.bias(SEED, 40 + l, N)
        dev.append(DevLayer(w, s_w, b, bits))
        layers.append(dict(M=M, N=N, K=K, bits=bits, w=w, s_w=s_w, bias=b))
    T, kept, bins = 9, [0, 4, 8], [8, 5, 3]
    xs = [[synth.activations(SEED, 40 + l, t, L["M"], L["K"], 1.0, n_out=max(1, L["K"] // 100))
           for l, L in enumerate(layers)] for t in kept]
    plan = B.dp_plan_create([d.w for d in dev], [L["M"] for L in layers], B.DP_FLAG_GROUP_SMALL_M)
    try:
        B.dp_plan_set_daq(plan, 99900, T, bins)
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        nL, nS = len(layers), len(kept)
        xd = [[to_dev_bf16(xs[i][l]) for l in range(nL)] for i in range(nS)]
        yd = [[torch.full((L["M"], L["N"]), float("nan"), dtype=torch.bfloat16, device="cuda")
               for L in layers] for _ in range(nS)]
        xp = B.ptr_array([xd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        yp = B.ptr_array([yd[i][l].data_ptr() for i in range(nS) for l in range(nL)])
        B.dp_plan_run(plan, kept, 0, xp, yp, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for i, t in enumerate(kept):
            bits = bins[min(2, 3 * t // T)]
            for l, L in enumerate(layers):
                q, s_a, _ = oracle.daq_robust(xs[i][l], oracle.clip_rank("99.9", L["K"]), bits)
                ref = oracle.epilogue(oracle.gemm_i32(q, L["w"]), s_a, L["s_w"], L["bias"])
                d = bf16_ulp_dist(bf16_to_np(yd[i][l]), ref)
                assert d.max() <= 1, (t, l, shapes[l], int(d.max()))
    finally:
        B.dp_plan_destroy(plan)


def test_plan_run_host_inputs():
    table, layers, dev = _mini_plan(tokens=128, batch=2, blocks=1)
    kept = [1, 3, 4]
    nL, nS = len(layers), len(kept)
    xs = [[synth.activations(SEED, l, t, L["M"], L["K"], 1.0, n_out=3) for l, L in enumerate(layers)]
          for t in kept]
    ref = oracle.plan_run(layers, kept, xs)
    plan = B.dp_plan_create([d.w for d in dev], [L["M"] for L in layers])
    try:
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        stage = torch.empty(2 * B.dp_plan_x_bytes(plan), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        xh = [[torch.from_numpy(xs[i][l].view(np.int16).copy()).pin_memory() for l in range(nL)] for i in range(nS)]
        yd = [torch.empty((L["M"], L["N"]), dtype=torch.bfloat16, device="cuda") for L in layers]
        last = nL - 2  # fc2 of the block
        yh = [torch.empty((layers[last]["M"], layers[last]["N"]), dtype=torch.bfloat16).pin_memory()
              for _ in range(nS)]
        B.dp_plan_run_host(plan, kept, B.ptr_array([xh[i][l].data_ptr() for i in range(nS) for l in range(nL)]),
                           stage, B.ptr_array([t.data_ptr() for t in yd]), last,
                           B.ptr_array([t.data_ptr() for t in yh]), ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for i in range(nS):
            got = yh[i].view(torch.int16).numpy().view(np.uint16)
            assert bf16_ulp_dist(got, ref[i][last]).max() <= 1
    finally:
        B.dp_plan_destroy(plan)


def test_plan_errors():
    table, layers, dev = _mini_plan(tokens=128, batch=1, blocks=1)
    bad = B.make_weight(dev[0].qweight, dev[0].s_w, None, dev[0].N, dev[0].K, 7)
    with pytest.raises(B.DiffproError) as e:
        B.dp_plan_create([bad], [128])
    assert e.value.status == B.DP_ERR_BITS
    plan = B.dp_plan_create([dev[0].w], [128])
    try:
        small = torch.empty(256, dtype=torch.uint8, device="cuda")
        x = torch.zeros((128, dev[0].K), dtype=torch.bfloat16, device="cuda")
        y = torch.zeros((128, dev[0].N), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(B.DiffproError) as e:
            B.dp_plan_run(plan, [0], 0, B.ptr_array([x.data_ptr()]), B.ptr_array([y.data_ptr()]), small)
        assert e.value.status == B.DP_ERR_WORKSPACE
    finally:
        B.dp_plan_destroy(plan)


def test_phase_a_on_measured_latencies_matches_oracle_and_runs():
    """Algorithm 2 end to end on a small stack: c_lat(l, b) measured with the library's kernels, Phase A
    (library) equal to the oracle's on the same table, and the resulting bit plan and kept steps run by
    dp_plan_run against the oracle's layer outputs."""
    from paper_2511_11446_b200 import planner
    seed = synth.BASE_SEED + 21
    table = [("a", 256, 256, 128), ("b", 256, 128, 256), ("c", 16, 256, 128), ("a2", 256, 256, 128)]
    lat = planner.latency_table(table, reps=5)
    assert all(v > 0.5 and v < 5e4 for v in lat.values()), lat
    T = 10
    drift = [float(np.exp(-t / 3.0)) + 0.01 * ((t * 7) % 3) for t in range(T)]
    sens = [0.5, 2.0, 1.0, 0.1]
    full = T * sum(lat[(M, K, N, 8)] for (_, M, K, N) in table) + T * 5.0
    mem8 = sum(N * K + 6 * N for (_, M, K, N) in table)
    B_lat = full - 22.0  # reachable by dropping steps (these small layers cost about the same at every width)
    bits, kept, totals, ok = planner.joint_plan(table, lat, sens, drift, 5.0, B_lat, 0.7 * mem8)
    options = [[(b, T * lat[(M, K, N, b)], N * K * b / 8 + 6 * N) for b in (8, 4, 3)] for (_, M, K, N) in table]
    o_bits, o_kept, o_tot, o_ok = oracle.phase_a(drift, [5.0] * T, options, sens, B_lat, 0.7 * mem8, 0.2, 1e-6)
    assert bits == o_bits and kept == [t for t in range(T) if o_kept[t]] and ok == o_ok and ok
    assert totals[1] <= 0.7 * mem8 and set(kept) >= {8, 9}
    # deploy (Phase B) under the plan
    Ls, Ws = [], []
    for l, (name, M, K, N) in enumerate(table):
        w, s_w = synth.weights(seed, l, N, K, bits[l])
        b = synth.bias(seed, l, N)
        Ls.append(DevLayer(w, s_w, b, bits[l]))
        Ws.append((w, s_w, b))
    plan = B.dp_plan_create([L.w for L in Ls], [M for (_, M, K, N) in table], 0)
    try:
        xs = [[synth.activations(seed, l, t, M, K, synth.sigma_t(t, T), n_out=2) for l, (_, M, K, N) in enumerate(table)]
              for t in kept]
        xd = [[to_dev_bf16(x) for x in row] for row in xs]
        ys = [[torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for (_, M, K, N) in table] for _ in kept]
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.dp_plan_run(plan, kept, 0, B.ptr_array([t.data_ptr() for row in xd for t in row]),
                      B.ptr_array([t.data_ptr() for row in ys for t in row]), ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        for i in range(len(kept)):
            for l, (w, s_w, b) in enumerate(Ws):
                ref = oracle.wq_linear(xs[i][l], oracle.pack(w, bits[l]), s_w, b, bits[l])
                assert bf16_ulp_dist(bf16_to_np(ys[i][l]), ref).max() <= 1
    finally:
        B.dp_plan_destroy(plan)


def test_chained_layers_whose_input_is_an_earlier_output():
    """A plan whose layer l + 1 reads the buffer layer l writes (x of one aliasing y of the other): the
    L2 hints a GEMM gives for the next layer's input must not let anything be read before its turn.
    Three chained linears over two steps, against the oracle's chain, several times in a row."""
    M, dims, bits = 1024, (384, 512, 256, 384), (8, 4, 3)
    ws_, dev, lay = [], [], []
    for l in range(3):
        K, N = dims[l], dims[l + 1]
        w, s_w = synth.weights(SEED + 50, l, N, K, bits[l])
        b = synth.bias(SEED + 50, l, N)
        dev.append(DevLayer(w, s_w, b, bits[l]))
        lay.append((oracle.pack(w, bits[l]), s_w, b, bits[l]))
    steps = [3, 7]
    x0 = [synth.activations(SEED + 50, 0, t, M, dims[0], 1.0, n_out=4) for t in steps]
    want = []
    for i in range(len(steps)):
        h, outs = x0[i], []
        for pw, s_w, b, bt in lay:
            h = oracle.wq_linear(h, pw, s_w, b, bt)
            outs.append(h)
        want.append(outs)
    plan = B.dp_plan_create([d.w for d in dev], [M] * 3)
    try:
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for rep in range(3):
            xd = [to_dev_bf16(x0[i]) for i in range(len(steps))]
            yd = [[torch.full((M, dims[l + 1]), float("nan"), dtype=torch.bfloat16, device="cuda") for l in range(3)]
                  for _ in steps]
            xp = B.ptr_array([(xd[i] if l == 0 else yd[i][l - 1]).data_ptr() for i in range(len(steps)) for l in range(3)])
            yp = B.ptr_array([yd[i][l].data_ptr() for i in range(len(steps)) for l in range(3)])
            B.dp_plan_run(plan, steps, 0, xp, yp, ws, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            for i in range(len(steps)):
                for l in range(3):
                    assert np.array_equal(bf16_to_np(yd[i][l]), want[i][l]), (rep, i, l)
    finally:
        B.dp_plan_destroy(plan)
