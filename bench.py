#!/usr/bin/env python
"""Benchmark of the DiffPro quantized-linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload (config.workload = "c4"): the whole DiT-XL/2 linear stack (28 blocks x {qkv, proj, fc1, fc2,
adaLN} = 140 quantized linears, mixed {3,4,8}-bit plan) executed by dp_plan_run over 25 retained of 50
timesteps at batch 8, 256 px (M = 2048 tokens; adaLN M = 8). One bench "step" = one dp_plan_run over
the full retained schedule = 3500 quantized linears (DAQ -> unpack -> INT8 GEMM -> dequant each).
`value` = int8 TOPS = 2*M*N*K summed over all calls / time; `us_per_dit_step` = time per denoising
timestep (140 linears). With N > 1 GPUs every rank runs the same-size workload on its own batch
(rows shard with no collective; weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused DAQ+WbA8 linear int8 TOPS (dp_plan_run, DiT-XL/2 linear stack)"
UNIT = "TOPS"
NOMINAL_INT8_TOPS = 4500.0
# dram__bytes_read.sum + dram__bytes_write.sum of one whole layer at M = 2048 (its DAQ launch, which for
# packed layers also expands the weights, plus its GEMM launch), per (shape, weight bits), from the ncu
# capture summarised in profiles/layer_dram_traffic_M2048.txt. None = no capture of the current kernels.
LAYER_DRAM_BYTES = {("qkv", 8): 22796480, ("qkv", 4): 21250107, ("qkv", 3): 20888222,
                    ("proj", 8): 10673745, ("proj", 4): 10187587, ("proj", 3): 10219431,
                    ("fc1", 8): 28953344, ("fc1", 4): 27161833, ("fc1", 3): 26080140,
                    ("fc2", 8): 29405184, ("fc2", 4): 25559239, ("fc2", 3): 24797924}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons, pw = [], [], set(), []
        for line in out.splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(pw), "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
def oracle_sample(seconds_target=15.0):
    """The CPU oracle, as it stands, on a bounded sample of the workload: the first layers of the
    stack (in plan order, their planned bit-widths) at the last retained timestep, as many as fit
    the time target. Returns (tops, seconds, description, cores)."""
    import oracle
    from paper_2511_11446_b200 import synth
    seed = synth.BASE_SEED + 4
    table = synth.dit_layers(8, 256)
    bits = synth.bit_plan(seed, len(table))
    t = synth.kept_timesteps(seed)[-1]

    def make(l, rows=None):
        _, M, K, N = table[l]
        M = M if rows is None else min(M, rows)
        w, s_w = synth.weights(seed, l, N, K, bits[l])
        x = synth.activations(seed, l, t, M, K, synth.sigma_t(t, 50), n_out=max(1, K // 100))
        return x, oracle.pack(w, bits[l]), s_w, synth.bias(seed, l, N), bits[l], 2.0 * M * N * K

    x, pw, s_w, b, bt, ops = make(0, rows=128)
    t0 = time.perf_counter(); oracle.wq_linear(x, pw, s_w, b, bt); rate = ops / (time.perf_counter() - t0)
    budget, chosen, tot = rate * seconds_target, [], 0.0
    for l in range(len(table)):
        o = 2.0 * table[l][1] * table[l][2] * table[l][3]
        if chosen and tot + o > budget:
            break
        chosen.append(l); tot += o
    secs = 0.0
    for l in chosen:
        x, pw, s_w, b, bt, ops = make(l)
        t0 = time.perf_counter(); oracle.wq_linear(x, pw, s_w, b, bt); secs += time.perf_counter() - t0
    desc = (f"layers 0..{chosen[-1]} of 140 (plan order, planned bits) of timestep {t}: "
            f"{tot / 1e9:.1f} of {sum(2.0 * M * N * K for _, M, K, N in table) * 25 / 1e9:.0f} GOP per plan run")
    return tot / secs / 1e12, secs, desc, oracle.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    vals, secs, desc, cores = [], [], "", 1
    for i in range(args.warmup + args.steps):
        tops, dt, desc, cores = oracle_sample(seconds_target=max(2.0, min(15.0, 120.0 / (args.warmup + args.steps))))
        if i >= args.warmup:
            vals.append(tops); secs.append(dt)
    v = sum(vals) / len(vals)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "c4", "note": "CPU oracle on a bounded sample per step: " + desc},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# --------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_2511_11446_b200 import binding as B, dist as D
    from paper_2511_11446_b200.workloads import DitStack
    from paper_2511_11446_b200 import synth

    rank, local_rank, world = D.init()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = measured_peaks()

    seed = D.rank_seed(synth.BASE_SEED + 4, rank)
    variants = None
    if args.load_variants:
        with open(args.load_variants) as f:
            variants = json.load(f)
    stack = DitStack(seed=seed, variants=variants)
    if args.daq_policy:  # e.g. 99900:8,6,4 = clip at the 99.9th percentile, 8/6/4 activation bits per time bin
        pe3, bins = args.daq_policy.split(":")
        B.dp_plan_set_daq(stack.plan, int(pe3), stack.T, [int(b) for b in bins.split(",")])
        stack.workspace = torch.empty(B.dp_plan_workspace(stack.plan), dtype=torch.uint8, device="cuda")
    if args.save_variants and rank == 0:
        with open(args.save_variants, "w") as f:
            json.dump(stack.layer_variants(), f)
    nL, nS = len(stack.table), len(stack.kept)
    ops_step = stack.ops_per_timestep() * nS
    graph = stack.capture()
    torch.cuda.synchronize()

    # ---- device-resident timing: K plan runs (graph replays), CUDA events on the launch stream ----
    # the clock sampler starts with the warm-up replays (the same work): nvidia-smi needs a few tenths
    # of a second to come up, more than a short timed region lasts
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        graph.replay()
    torch.cuda.synchronize()
    D.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.cudart().cudaProfilerStart()  # lets `ncu --profile-from-start off` see only the timed region
    e0.record()
    for _ in range(args.steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    torch.cuda.cudart().cudaProfilerStop()
    D.barrier()
    ms_total = D.max_over_ranks(e0.elapsed_time(e1), dev)
    clocks = sampler.stop()
    assert int(stack.status.item()) == 0, "a kernel reported DP_ERR_TIMEOUT"
    ms_per_step = ms_total / args.steps
    value = world * ops_step / (ms_per_step * 1e-3) / 1e12

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8", "data": "synthetic",
        "config": {"workload": "c4", "layers": nL, "retained_timesteps": nS, "of_timesteps": stack.T,
                   "M": 2048, "M_adaln": 8, "bit_plan_counts": {str(b): stack.bits.count(b) for b in (3, 4, 8)},
                   "parallelism": f"rows x{world} (no collective)", "l2": "inputs+weights per timestep (>1.1 GB) exceed L2",
                   "launch": "one CUDA graph per plan run",
                   "daq_policy": args.daq_policy or "absmax, 8 bits (the metric's definition)"},
        "us_per_dit_step": 1e3 * ms_per_step / nS,
        "roofline_step": {"ideal_us_per_dit_step_nominal": None},
        "gpu_launches": stack.launches_per_timestep() * nS * args.steps,
        "clocks": clocks,
    }

    if rank == 0 and args.timed_only:
        print(json.dumps(out))
    elif rank == 0:
        # ---- roofline of the dominant kernel (tcgen05 GEMM), timed alone with CUDA events ----
        mma_peak = measure_mma_peak()
        out["roofline"] = gemm_roofline(stack, peaks, mma_peak)
        # ideal time of a timestep: per layer max(ops / int8 peak, bytes / HBM); the int8 peak is the
        # larger of sustained bf16 x2 (the step is seconds of back-to-back work) and the measured
        # instruction ceiling
        int8_peak = max(2.0 * peaks["bf16_sustained"], mma_peak or 0.0)
        ideal = 0.0
        for l, (_, M, K, N) in enumerate(stack.table):
            ideal += max(2.0 * M * N * K / (int8_peak * 1e12), layer_alg_bytes(stack, l) / (peaks["hbm_gbs"] * 1e9))
        out["roofline_step"] = {"ideal_us_per_dit_step": ideal * 1e6, "frac": ideal * 1e6 / out["us_per_dit_step"],
                                "int8_peak_tops_used": int8_peak, "hbm_gbs_used": peaks["hbm_gbs"],
                                "peaks": peaks["source"]}
        out["mma_i8_peak_tops_measured"] = mma_peak
        out["roofline_hbm_kernels"] = hbm_kernel_rooflines(stack, peaks)
        out["roofline_large_m"] = large_m_rooflines(peaks, mma_peak)
        out["next_rows"] = next_row_timings(peaks)
        out["e2e"] = e2e(stack, ops_step, world)
        tops, dt, desc, cores = oracle_sample()
        out["cpu_baseline"] = {"value": tops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                               "seconds": dt}
        print(json.dumps(out))
    stack.close()
    D.barrier()


def layer_alg_bytes(stack, l):
    """Bytes the method itself must move for layer l: X bf16, packed W, s_w + bias, Y bf16."""
    _, M, K, N = stack.table[l]
    return 2 * M * K + stack.layers[l].packed_bytes() + 6 * N + 2 * M * N


def gemm_roofline(stack, peaks, mma_peak):
    """The dominant kernel family (the tcgen05 GEMMs) timed without the rest of the path: the 112
    GEMM launches of one timestep, each with the kernel variant the plan chose for its layer, on
    pre-quantized activations (so no DAQ launch in between), captured in one CUDA graph and timed
    with CUDA events on the replay stream. One timestep's operands (0.4 GB of int8 activations,
    0.4 GB of weights, 1.1 GB of outputs) exceed L2, so every launch streams from HBM. A layer the
    plan runs in the unpack-first form launches the 8-bit kernel on an int8 copy of its weights:
    here that copy is generated directly (same seeded values), so the launch is that GEMM alone."""
    import collections
    import torch
    from paper_2511_11446_b200 import binding as B, synth_cuda
    x0 = stack.x[0]
    idx = [l for l, (_, M, K, N) in enumerate(stack.table) if M > 32]
    qs, sas, flags, variants, weights, keep = {}, {}, {}, collections.Counter(), {}, []
    for l in idx:
        _, M, K, N = stack.table[l]
        qs[l] = torch.empty((M, K), dtype=torch.int8, device="cuda")
        sas[l] = torch.empty(M, dtype=torch.float32, device="cuda")
        B.dp_daq_quantize(x0[l], M, K, K, qs[l], K, sas[l])
        v = B.dp_plan_layer_variant(stack.plan, l)
        flags[l] = B.variant_flags(v)
        weights[l] = stack.layers[l].w
        if v["unpack_first"]:
            w8, _ = synth_cuda.weights(stack.seed, l, N, K, stack.bits[l])
            keep.append(w8)
            weights[l] = B.make_weight(w8, stack.layers[l].s_w, stack.layers[l].bias, N, K, 8)
            flags[l] &= ~B.DP_FLAG_UNPACK_FIRST
        variants[("as" if v["weight_stationary"] == 2 else "ws" if v["weight_stationary"] else
                  "pair" if v["cta_group"] == 2 else "single") + str(v["tile_n"])
                 + ("+unpack_first" if v["unpack_first"] else "")] += 1

    def run():
        for l in idx:
            _, M, K, N = stack.table[l]
            B.dp_wq_linear(weights[l], qs[l], K, sas[l], M, stack.y[l], N, None, None, stack.status, flags[l])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        run()
    times = []
    for it in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = statistics.median(times[1:])
    ops = sum(2.0 * stack.table[l][1] * stack.table[l][2] * stack.table[l][3] for l in idx)
    achieved = ops / (ms * 1e-3) / 1e12
    # Denominator: the larger of (measured bf16 burst x the nominal int8:bf16 ratio of 2) and this
    # library's own operand-resident kind::i8 instruction ceiling measured in the same run.
    bf16x2 = 2.0 * peaks["bf16"]
    peak = max(bf16x2, mma_peak or 0.0)
    alg = sum(layer_alg_bytes(stack, l) for l in idx) / len(idx)
    traffic = None
    if LAYER_DRAM_BYTES is not None:
        traffic = sum(LAYER_DRAM_BYTES[(stack.table[l][0].split(".")[1], stack.bits[l])] for l in idx) / len(idx)
    return {"kernel": "gemm_i8_kernel (tcgen05 kind::i8), the 112 launches of one timestep",
            "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TOPS", "frac": achieved / peak,
            "peak_note": f"max of {peaks['source']} bf16 burst x2 = {bf16x2:.0f} (nominal int8:bf16 ratio; the file has "
                         f"no int8 row) and the kind::i8 instruction ceiling measured in this run = "
                         f"{mma_peak or 0.0:.0f}; sustained bf16 x2 = {2.0 * peaks['bf16_sustained']:.0f}; "
                         f"nominal dense int8 {NOMINAL_INT8_TOPS:.0f}",
            "frac_of_bf16x2": achieved / bf16x2, "frac_of_nominal": achieved / NOMINAL_INT8_TOPS, "launches": len(idx),
            "avg_launch_us": 1e3 * ms / len(idx), "variants": dict(variants),
            "traffic": traffic, "traffic_note": "DRAM bytes of a whole layer (DAQ + GEMM launches, reads + writes), "
                                                "mean over the step's 112 layers; algorithmic bytes beside it",
            "algorithmic_bytes_per_layer": alg}


def hbm_kernel_rooflines(stack, peaks):
    """The HBM-bound kernels of the path against the measured copy bandwidth: (a) the adaLN
    modulation linears of one timestep (28 layers, M = batch, mixed bits) as the plan runs them, one
    grouped launch, bytes = packed weights + inputs + outputs; (b) dp_daq_quantize at M = 32768."""
    import torch
    from paper_2511_11446_b200 import binding as B, synth_cuda, synth

    def graph_time(fn, reps=5):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts[1:]) * 1e-3

    out = {}
    idx = [l for l, (_, M, K, N) in enumerate(stack.table) if M <= 32]
    plan = B.dp_plan_create([stack.layers[l].w for l in idx], [stack.table[l][1] for l in idx],
                            B.DP_FLAG_GROUP_SMALL_M)
    try:
        ws = torch.empty(B.dp_plan_workspace(plan), dtype=torch.uint8, device="cuda")
        xp = B.ptr_array([stack.x[0][l].data_ptr() for l in idx])
        yp = B.ptr_array([stack.y[l].data_ptr() for l in idx])
        # four passes per graph replay: the 133 MB of packed weights exceed L2, so each pass streams
        # them from HBM again
        def passes():
            for _ in range(4):
                B.dp_plan_run(plan, [0], 0, xp, yp, ws, stack.status, flags=B.DP_PLAN_SAME_X | B.DP_PLAN_SAME_Y)
        t = graph_time(passes) / 4
        by = sum(stack.layers[l].packed_bytes() + 6 * stack.table[l][3] + 2 * stack.table[l][1] * (stack.table[l][2] + stack.table[l][3])
                 for l in idx)
        out["adaln_group"] = {"layers": len(idx), "bytes": by, "us": t * 1e6, "achieved": by / t / 1e9,
                              "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": by / t / 1e9 / peaks["hbm_gbs"]}
    finally:
        B.dp_plan_destroy(plan)
    for K in (1152, 4608):
        M = 32768
        x = synth_cuda.activations(synth.BASE_SEED, 0, 0, M, K, 1.0, n_out=K // 100)
        q = torch.empty((M, K), dtype=torch.int8, device="cuda")
        sa = torch.empty(M, dtype=torch.float32, device="cuda")
        x2 = x.clone(); q2 = torch.empty_like(q)  # 2 sets: 2 x (75 + 38) MB or 2 x (302 + 151) MB, past L2
        def run():
            B.dp_daq_quantize(x, M, K, K, q, K, sa)
            B.dp_daq_quantize(x2, M, K, K, q2, K, sa)
        t = graph_time(run) / 2
        by = 3 * M * K + 4 * M
        out[f"daq_M32768_K{K}"] = {"bytes": by, "us": t * 1e6, "achieved": by / t / 1e9, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": by / t / 1e9 / peaks["hbm_gbs"]}
        rank = B.dp_clip_rank(99900, K)  # the equation's percentile clip, 8-bit codes

        def run_robust():
            B.dp_daq_quantize_robust(x, M, K, K, q, K, sa, rank, 8)
            B.dp_daq_quantize_robust(x2, M, K, K, q2, K, sa, rank, 8)
        t = graph_time(run_robust) / 2
        out[f"daq_robust_p99.9_M32768_K{K}"] = {"bytes": by, "us": t * 1e6, "achieved": by / t / 1e9,
                                                 "peak": peaks["hbm_gbs"], "unit": "GB/s", "clip_rank": rank,
                                                 "frac": by / t / 1e9 / peaks["hbm_gbs"]}
        del x, x2, q, q2
    return out


def large_m_rooflines(peaks, mma_peak):
    """Config 5 (M = 32768 tokens): the four block shapes at 3, 4 and 8 weight bits, the whole layer
    (DAQ + weight expansion + GEMM, default dispatch of dp_wq_linear) and the GEMM alone on
    pre-quantized activations, graph-timed with operand sets rotated past L2. Fractions: against the
    per-layer roofline max(ops / int8 peak, algorithmic bytes / measured HBM bandwidth) for the
    layer, against the int8 peak for the GEMM alone (same denominator as `roofline`)."""
    from paper_2511_11446_b200 import sweep
    int8_peak = max(2.0 * peaks["bf16"], mma_peak or 0.0)
    rows = []
    for name, K, N in sweep.SHAPES:
        for bits in (3, 4, 8):
            r = sweep.time_shape(name, 32768, K, N, bits, dict(peaks, bf16=int8_peak / 2.0), iters=8)
            rows.append({"layer": name, "bits": bits, "layer_us": r["layer_us"], "layer_tops": r["layer_tops"],
                         "layer_frac_of_roofline": r["layer_frac"], "bound": r["bound"], "gemm_us": r["gemm_us"],
                         "gemm_tops": r["gemm_tops"], "gemm_frac_of_int8_peak": r["gemm_frac_int8_peak"],
                         "gemm_frac_of_nominal": r["gemm_tops"] / NOMINAL_INT8_TOPS})
    return {"M": 32768, "int8_peak_tops_used": int8_peak, "hbm_gbs_used": peaks["hbm_gbs"], "shapes": rows}


def next_row_timings(peaks):
    """The rows beyond the per-channel W{3,4,8}A8 path, whole layers at M = 2048, graph-timed with
    operands rotated past L2: group-wise weight scales (Step 2's storage format; g = 128 and 32, 4-bit,
    with and without zero-points) and 16-bit pass-through layers (bf16, fp32 accumulation; fraction
    against the measured bf16 tensor rate), and the gated residual add taken into the epilogue of the two
    layers that feed the token stream, beside the same layer without it; LayerNorm + adaLN modulation
    taken into DAQ beside plain DAQ of the same tokens (M = 2048 and 32768)."""
    from paper_2511_11446_b200 import sweep
    out = {"M": 2048, "grouped": [], "passthrough_bf16": [], "gated_residual": [],
           "ln_modulate_daq": [sweep.time_ln_daq(2048, 1152, peaks), sweep.time_ln_daq(32768, 1152, peaks)]}
    for name, K, N in sweep.SHAPES:
        if N == 1152:  # the two layers of a DiT block that feed the token stream: proj and fc2
            r = sweep.time_residual(name, 2048, K, N, 4, peaks)
            plain = sweep.time_shape(name, 2048, K, N, 4, peaks, only="layer")
            out["gated_residual"].append({"layer": name, "bits": 4, "layer_us": r["layer_us"],
                                          "plain_layer_us": plain["layer_us"]})
        for g, zp in ((128, False), (128, True), (32, False)):
            r = sweep.time_grouped(name, 2048, K, N, 4, g, zp, peaks)
            out["grouped"].append({k: r[k] for k in ("layer", "bits", "group_size", "zero_points", "layer_us", "layer_tops")})
        r = sweep.time_shape(name, 2048, K, N, 16, peaks, only="layer")
        out["passthrough_bf16"].append({"layer": name, "layer_us": r["layer_us"], "tflops": r["layer_tops"],
                                        "frac_of_measured_bf16": r["layer_tops"] / peaks["bf16"]})
    return out


def measure_mma_peak():
    import torch
    from paper_2511_11446_b200 import probe
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    iters = 20000
    probe.dp_probe_mma_i8(sms, 2000, 256, st)
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        probe.dp_probe_mma_i8(sms, iters, 256, st)
        e1.record()
        torch.cuda.synchronize()
        best = max(best, 2.0 * 128 * 256 * 128 * iters * sms / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    return best if int(st.item()) == 0 else None


def e2e(stack, ops_step, world):
    """Same plan run through dp_plan_run_host: every timestep's inputs are copied from pinned host
    memory inside the timed region and the last block's fc2 output is read back per timestep."""
    import psutil
    import torch
    from paper_2511_11446_b200 import binding as B
    nL, nS = len(stack.table), len(stack.kept)
    xbytes = sum(t.numel() * 2 for t in stack.x[0])
    distinct = psutil.virtual_memory().available > 3 * xbytes * nS
    n_host = nS if distinct else 1
    xh = [[torch.empty(t.shape, dtype=torch.bfloat16, pin_memory=True) for t in stack.x[0]] for _ in range(n_host)]
    for i in range(n_host):
        for l in range(nL):
            xh[i][l].copy_(stack.x[i][l])
    last = nL - 2
    M, N = stack.table[last][1], stack.table[last][3]
    yh = [torch.empty((M, N), dtype=torch.bfloat16, pin_memory=True) for _ in range(nS)]
    stage = torch.empty(2 * B.dp_plan_x_bytes(stack.plan), dtype=torch.uint8, device="cuda")
    xp = B.ptr_array([xh[i][l].data_ptr() for i in range(n_host) for l in range(nL)])
    yp = B.ptr_array([t.data_ptr() for t in stack.y])
    yhp = B.ptr_array([t.data_ptr() for t in yh])
    flags = 0 if distinct else B.DP_PLAN_SAME_X
    times = []
    for it in range(3):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.dp_plan_run_host(stack.plan, stack.kept, xp, stage, yp, last, yhp, stack.workspace, stack.status, flags)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = min(times[1:])
    return {"value": world * ops_step / (ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": xbytes * nS, "d2h_bytes_per_step": M * N * 2 * nS,
            "host_inputs": "distinct per timestep" if distinct else "one timestep's buffers re-copied every timestep"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", default=None, choices=["c1", "c2", "c3", "c4", "c5"],
                    help="per-shape timing table (one JSON line per layer shape and bit-width) instead of the plan run")
    ap.add_argument("--bits", default="3,4,8")
    ap.add_argument("--layers", default=None, help="comma list out of qkv,proj,fc1,fc2,adaln")
    ap.add_argument("--only", default=None, choices=["layer", "gemm", "daq"])
    ap.add_argument("--iters", type=int, default=None)
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0, help="dp_wq_linear tuning flags for --sweep")
    ap.add_argument("--group", type=int, default=0, help="--sweep with group-wise weight scales of this group size")
    ap.add_argument("--zero-points", action="store_true", help="--sweep --group with zero-points")
    ap.add_argument("--save-variants", default=None,
                    help="write the per-layer kernel variants the autotuner chose to this JSON file")
    ap.add_argument("--load-variants", default=None,
                    help="apply per-layer kernel variants from this JSON file instead of autotuning (a run "
                         "under a profiler times variants differently, so profiles reuse a plain run's choice)")
    ap.add_argument("--daq-policy", default=None,
                    help="P:a,b,c = run the plan under dp_plan_set_daq(P/1000 percent clip, activation bits of the "
                         "three time bins); default: the absmax, 8-bit rule the headline metric is defined on")
    ap.add_argument("--timed-only", action="store_true",
                    help="only the timed plan run (no roofline, side measurements, end-to-end or CPU legs): for runs "
                         "under a profiler; its line is not a benchmark result")
    ap.add_argument("--hbm-kernels", action="store_true",
                    help="time only the HBM-bound kernels (grouped adaLN launch, DAQ at M=32768) and print their rooflines")
    args = ap.parse_args()
    if args.hbm_kernels:
        import torch
        from paper_2511_11446_b200 import synth
        from paper_2511_11446_b200.workloads import DitStack
        torch.cuda.set_device(0)
        from paper_2511_11446_b200 import binding as B
        stack = DitStack(seed=synth.BASE_SEED + 4, flags=B.DP_FLAG_GROUP_SMALL_M)  # no autotuning needed here
        print(json.dumps(hbm_kernel_rooflines(stack, measured_peaks())))
        return
    if args.sweep:
        import torch
        from paper_2511_11446_b200 import sweep
        torch.cuda.set_device(0)
        sweep.run(args.sweep, [int(b) for b in args.bits.split(",")], measured_peaks(), only=args.only,
                  layers=args.layers.split(",") if args.layers else None, iters=args.iters, flags=args.flags,
                  group=args.group, zeros=args.zero_points)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
