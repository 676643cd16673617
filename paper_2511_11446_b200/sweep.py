"""Per-shape timing of the quantized linear on one GPU (used by ``bench.py --sweep``).

For every (layer shape, weight bit-width) of a workload this times, with CUDA events on the launch
stream, (a) the whole layer through dp_wq_linear (DAQ inside the call), (b) the GEMM alone on
pre-quantized activations and (c) dp_daq_quantize alone. Buffers rotate over enough copies to exceed
the L2 cache, so every launch streams its operands from HBM as it does inside a plan run.
Only input preparation and bookkeeping live here; the arithmetic is in the CUDA library.
"""
from __future__ import annotations

import json

import torch

from . import binding as B
from . import synth, synth_cuda
from .workloads import DevWeights

L2_BYTES = 126 << 20
SHAPES = (("qkv", synth.HIDDEN, 3 * synth.HIDDEN), ("proj", synth.HIDDEN, synth.HIDDEN),
          ("fc1", synth.HIDDEN, synth.MLP), ("fc2", synth.MLP, synth.HIDDEN))
WORKLOADS = {"c1": (256, 1), "c2": (2048, 8), "c3": (4096, 16), "c4": (2048, 8), "c5": (32768, 32)}


def alg_bytes(M, K, N, bits):
    """Bytes the method itself must move for one layer: X bf16, packed W, s_w, bias, Y bf16."""
    return 2 * M * K + N * K * bits // 8 + 6 * N + 2 * M * N


def _time(fn, n_sets, iters, warmup=3):
    """us per launch of fn(set_index): `iters` launches captured in one CUDA graph (so the host's
    launch cost is not in the number), replayed after a warm-up replay."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(min(warmup, n_sets)):
            fn(i % n_sets)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for i in range(iters):
            fn(i % n_sets)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / iters


def time_grouped(name, M, K, N, bits, g, zeros, peaks, seed=synth.BASE_SEED + 5, iters=None):
    """Whole layer with group-wise weight scales (group size g, optional zero-points), graph-timed like
    time_shape; the scales are seeded positive numbers (their values do not change the work)."""
    per_set = 2 * M * K + M * K + 2 * M * N + N * K * bits // 8
    n_sets = max(2, min(24, -(-2 * L2_BYTES // per_set)))
    iters = iters or max(10, min(200, int(2e9 // per_set)))
    iters = -(-iters // n_sets) * n_sets
    Ws = [DevWeights(seed, s, N, K, bits) for s in range(n_sets)]
    gen = torch.Generator(device="cuda").manual_seed(seed)
    sc = [torch.rand((N, K // g), generator=gen, device="cuda") * 1e-2 + 1e-4 for _ in range(n_sets)]
    zs = [torch.randint(0, 1 << bits, (N, K // g), generator=gen, device="cuda", dtype=torch.uint8) if zeros else None
          for _ in range(n_sets)]
    ws_ = [B.make_weight(Ws[s].qweight, sc[s], Ws[s].bias, N, K, bits, g, zs[s]) for s in range(n_sets)]
    xs = [synth_cuda.activations(seed, s, 0, M, K, 1.0, n_out=max(1, K // 100)) for s in range(n_sets)]
    ys = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(n_sets)]
    ws = torch.empty(B.dp_wq_linear_workspace_grouped(M, ws_[0]), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t = _time(lambda s: B.dp_wq_linear(ws_[s], xs[s], K, None, M, ys[s], N, ws, None, status, 0), n_sets, iters)
    assert int(status.item()) == 0, "a kernel reported DP_ERR_TIMEOUT"
    ops = 2.0 * M * N * K
    by = alg_bytes(M, K, N, bits) + (4 + (1 if zeros else 0)) * N * (K // g) - 4 * N
    t_ideal = max(ops / (2.0 * peaks["bf16"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e6
    return {"layer": name, "M": M, "K": K, "N": N, "bits": bits, "group_size": g, "zero_points": bool(zeros),
            "layer_us": t, "layer_tops": ops / t / 1e6, "ideal_us": t_ideal, "layer_frac": t_ideal / t}


def time_ln_daq(M, K, peaks, rows_per_sample=256, seed=synth.BASE_SEED + 5, iters=None):
    """LayerNorm + adaLN modulation + DAQ in one pass against plain DAQ of the same tokens (both read
    2 bytes and write 1 byte per element), graph-timed with buffers rotated past L2."""
    per_set = 3 * M * K
    n_sets = max(2, min(24, -(-2 * L2_BYTES // per_set)))
    iters = iters or max(10, min(200, int(2e9 // per_set)))
    iters = -(-iters // n_sets) * n_sets
    xs = [synth_cuda.activations(seed, s, 0, M, K, 1.0, n_out=max(1, K // 100)) for s in range(n_sets)]
    qs = [torch.empty((M, K), dtype=torch.int8, device="cuda") for _ in range(n_sets)]
    sas = [torch.empty(M, dtype=torch.float32, device="cuda") for _ in range(n_sets)]
    S = -(-M // rows_per_sample)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    shift = (torch.randn((S, K), generator=gen, device="cuda") * 0.3).to(torch.bfloat16)
    scale = (torch.randn((S, K), generator=gen, device="cuda") * 0.3).to(torch.bfloat16)
    t_ln = _time(lambda s: B.dp_ln_modulate_daq(xs[s], M, K, K, shift, scale, rows_per_sample, 1e-6, qs[s], K, sas[s]),
                 n_sets, iters)
    t_daq = _time(lambda s: B.dp_daq_quantize(xs[s], M, K, K, qs[s], K, sas[s]), n_sets, iters)
    by = 3 * M * K + 4 * M
    return {"M": M, "K": K, "ln_modulate_daq_us": t_ln, "daq_us": t_daq, "bytes": by,
            "frac_of_hbm": by / (t_ln * 1e-6) / 1e9 / peaks["hbm_gbs"]}


def time_residual(name, M, K, N, bits, peaks, rows_per_gate=1024, seed=synth.BASE_SEED + 5, iters=None):
    """Whole layer with the gated residual in its epilogue (x <- x + gate * layer(h), written over x),
    graph-timed like time_shape; the stream adds 2*M*N bytes of reads to the layer's algorithmic bytes."""
    per_set = 2 * M * K + M * K + 4 * M * N + N * K * bits // 8
    n_sets = max(2, min(24, -(-2 * L2_BYTES // per_set)))
    iters = iters or max(10, min(200, int(2e9 // per_set)))
    iters = -(-iters // n_sets) * n_sets
    Ws = [DevWeights(seed, s, N, K, bits) for s in range(n_sets)]
    xs = [synth_cuda.activations(seed, s, 0, M, K, 1.0, n_out=max(1, K // 100)) for s in range(n_sets)]
    rs = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(n_sets)]
    gates = [torch.full((-(-M // rows_per_gate), N), 0.5, dtype=torch.bfloat16, device="cuda") for _ in range(n_sets)]
    fl = B.DP_FLAG_FORCE_MMA | B.DP_FLAG_UNPACK_FIRST
    nws = B.dp_wq_linear_workspace(M, N, K, bits, fl)
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t = _time(lambda s: B.dp_wq_linear_residual(Ws[s].w, xs[s], K, M, rs[s], N, gates[s], rows_per_gate, rs[s], N, ws,
                                                nws, status, 0), n_sets, iters)
    assert int(status.item()) == 0, "a kernel reported DP_ERR_TIMEOUT"
    ops = 2.0 * M * N * K
    by = alg_bytes(M, K, N, bits) + 2 * M * N
    t_ideal = max(ops / (2.0 * peaks["bf16"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e6
    return {"layer": name, "M": M, "K": K, "N": N, "bits": bits, "layer_us": t, "layer_tops": ops / t / 1e6,
            "ideal_us": t_ideal, "layer_frac": t_ideal / t}


def time_shape(name, M, K, N, bits, peaks, seed=synth.BASE_SEED + 5, iters=None, only=None, flags=0):
    per_set = 2 * M * K + M * K + 2 * M * N + N * K * bits // 8
    n_sets = max(2, min(24, -(-2 * L2_BYTES // per_set)))
    iters = iters or max(10, min(200, int(2e9 // per_set)))
    iters = -(-iters // n_sets) * n_sets
    Ws = [DevWeights(seed, s, N, K, bits) for s in range(n_sets)]
    xs = [synth_cuda.activations(seed, s, 0, M, K, 1.0, n_out=max(1, K // 100)) for s in range(n_sets)]
    qs = [torch.empty((M, K), dtype=torch.int8, device="cuda") for _ in range(n_sets)]
    sas = [torch.empty(M, dtype=torch.float32, device="cuda") for _ in range(n_sets)]
    ys = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(n_sets)]
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, bits, flags), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for s in range(n_sets):
        B.dp_daq_quantize(xs[s], M, K, K, qs[s], K, sas[s])
    out = {"layer": name, "M": M, "K": K, "N": N, "bits": bits, "buffer_sets": n_sets, "iters": iters}
    ops, by = 2.0 * M * N * K, alg_bytes(M, K, N, bits)
    int8_peak = 2.0 * peaks["bf16"]
    t_ideal = max(ops / (int8_peak * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e6
    out["ideal_us"] = t_ideal
    out["bound"] = "tensor" if ops / (int8_peak * 1e12) > by / (peaks["hbm_gbs"] * 1e9) else "hbm"
    if only in (None, "layer"):
        t = _time(lambda s: B.dp_wq_linear(Ws[s].w, xs[s], K, None, M, ys[s], N, ws, None, status, flags),
                  n_sets, iters)
        out.update(layer_us=t, layer_tops=ops / t / 1e6, layer_gbs=by / t / 1e3, layer_frac=t_ideal / t)
    if only in (None, "gemm") and bits != 16:
        t = _time(lambda s: B.dp_wq_linear(Ws[s].w, qs[s], K, sas[s], M, ys[s], N, ws, None, status, flags),
                  n_sets, iters)
        out.update(gemm_us=t, gemm_tops=ops / t / 1e6, gemm_frac_int8_peak=ops / t / 1e6 / int8_peak)
    if only in (None, "daq"):
        t = _time(lambda s: B.dp_daq_quantize(xs[s], M, K, K, qs[s], K, sas[s]), n_sets, iters)
        out.update(daq_us=t, daq_gbs=(3 * M * K + 4 * M) / t / 1e3,
                   daq_frac_hbm=(3 * M * K + 4 * M) / t / 1e3 / peaks["hbm_gbs"])
    assert int(status.item()) == 0, "a kernel reported DP_ERR_TIMEOUT"
    return out


def run(workload, bits_list, peaks, only=None, layers=None, iters=None, flags=0, emit=print, group=0, zeros=False):
    M, batch = WORKLOADS[workload]
    rows = []
    for name, K, N in SHAPES:
        if layers and name not in layers:
            continue
        for bits in bits_list:
            if group:
                r = time_grouped(name, M, K, N, bits, group, zeros, peaks, iters=iters)
                r["workload"] = workload
                rows.append(r)
                emit(json.dumps(r))
                torch.cuda.empty_cache()
                continue
            r = time_shape(name, M, K, N, bits, peaks, iters=iters, only=only, flags=flags)
            r["workload"] = workload
            rows.append(r)
            emit(json.dumps(r))
            torch.cuda.empty_cache()
    if group:
        return rows
    if not layers or "adaln" in layers:
        for bits in bits_list:
            r = time_shape("adaln", batch, synth.HIDDEN, synth.ADALN, bits, peaks, iters=iters, only="layer",
                           flags=flags)
            r["workload"] = workload
            rows.append(r)
            emit(json.dumps(r))
    return rows
