"""Synthetic DiT-XL/2 workloads resident on the GPU, built from the seeded generators.

`DitStack` is the whole linear stack of DiT-XL/2 (28 blocks x {qkv, proj, fc1, fc2, adaLN}) with a
per-layer bit plan from {3,4,8} and a retained-timestep schedule (25 of 50), as the deployed plan of
Algorithm 2 Phase B sees it. Inputs are regenerated per (layer, timestep) with std 0.5 + 2t/T and a
per-timestep 1 % outlier-channel set. Everything here is input preparation and bookkeeping; the
quantized-linear arithmetic is in the CUDA library.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synth, synth_cuda


class DevWeights:
    """One layer's constants on the device; integer weights come from the CUDA generator and are
    packed by the library's host packer."""

    def __init__(self, seed, layer, N, K, bits, with_bias=True):
        self.N, self.K, self.bits = N, K, bits
        w, s_w = synth_cuda.weights(seed, layer, N, K, 8 if bits == 16 else bits)
        if bits == 16:  # a pass-through layer: the dequantized 8-bit weights, rounded to bf16
            self.qweight = (w.float() * s_w[:, None]).to(torch.bfloat16)
        elif bits == 8:
            self.qweight = w
        else:
            packed = B.dp_pack_weights_host(w.cpu().numpy(), bits)
            self.qweight = torch.from_numpy(packed.view(np.uint8)).cuda()
        self.s_w = s_w
        self.bias = None
        if with_bias:
            self.bias = torch.from_numpy(synth.bias(seed, layer, N).view(np.int16)).cuda().view(torch.bfloat16)
        self.w = B.make_weight(self.qweight, self.s_w, self.bias, N, K, bits)

    def packed_bytes(self):
        return self.N * self.K * self.bits // 8


class DitStack:
    def __init__(self, seed=synth.BASE_SEED + 4, batch=8, tokens=256, blocks=synth.BLOCKS, T=50, keep=25,
                 bit_choices=(3, 4, 8), resident_steps=None,
                 flags=B.DP_FLAG_AUTOTUNE | B.DP_FLAG_GROUP_SMALL_M, variants=None):
        """variants: per-layer tuning flags from an earlier autotuned stack's layer_variants() (None
        entries: small-M layers); given, the plan applies them instead of timing variants itself."""
        if variants is not None:
            flags &= ~B.DP_FLAG_AUTOTUNE
        self.seed, self.T, self.flags = seed, T, flags
        self.table = synth.dit_layers(batch, tokens, blocks)
        self.bits = synth.bit_plan(seed, len(self.table), bit_choices)
        self.kept = synth.kept_timesteps(seed, T, keep, 0.2)
        self.layers = [DevWeights(seed, l, N, K, self.bits[l]) for l, (_, M, K, N) in enumerate(self.table)]
        self.Ms = [M for (_, M, K, N) in self.table]
        self.plan = B.dp_plan_create([L.w for L in self.layers], self.Ms, flags)
        if variants is not None:
            for l, f in enumerate(variants):
                if f is not None:
                    B.dp_plan_set_layer_flags(self.plan, l, f)
        self.workspace = torch.empty(B.dp_plan_workspace(self.plan), dtype=torch.uint8, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.y = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for (_, M, K, N) in self.table]
        n_res = len(self.kept) if resident_steps is None else resident_steps
        self.x = [[self.gen_input(l, t) for l in range(len(self.table))] for t in self.kept[:n_res]]
        torch.cuda.synchronize()

    def gen_input(self, l, t, out=None):
        _, M, K, _ = self.table[l]
        return synth_cuda.activations(self.seed, l, t, M, K, synth.sigma_t(t, self.T), n_out=max(1, K // 100),
                                      out=out)

    def host_input_rows(self, l, t, rows):
        """The same input rows regenerated on the host (for sampled oracle checks)."""
        _, M, K, _ = self.table[l]
        return synth.activations(self.seed, l, t, M, K, synth.sigma_t(t, self.T), n_out=max(1, K // 100),
                                 rows=rows)

    def layer_variants(self):
        """Per layer: the tuning flags naming the kernel variant the plan runs (None: small-M kernel)."""
        out = []
        for l in range(len(self.table)):
            v = B.dp_plan_layer_variant(self.plan, l)
            out.append(None if v["small_m"] else
                       B.variant_flags(v) & ~(B.DP_FLAG_FORCE_MMA | B.DP_FLAG_FORCE_SIMT))
        return out

    # ---- accounting ----
    def ops_per_timestep(self):
        return sum(2 * M * N * K for (_, M, K, N) in self.table)

    def alg_bytes_per_timestep(self):
        tot = 0
        for L, (_, M, K, N) in zip(self.layers, self.table):
            tot += 2 * M * K + L.packed_bytes() + 4 * N + 2 * N + 2 * M * N
        return tot

    def launches_per_timestep(self):
        """Kernel launches of this library per timestep: DAQ + GEMM per token linear; the small-M
        (adaLN) linears of a step share, per 32 of them, one grouped launch that also quantizes their
        tokens when the plan groups them (under a percentile / a-bit DAQ policy a second, small
        quantization launch goes in front of it)."""
        small = sum(1 for (_, M, K, N) in self.table if M <= 32)
        big = len(self.table) - small
        grouped = bool(self.flags & B.DP_FLAG_GROUP_SMALL_M)
        return 2 * big + (-(-small // 32) if grouped else small)

    # ---- execution ----
    def ptrs(self, n_steps=None):
        n_steps = len(self.x) if n_steps is None else n_steps
        xp = B.ptr_array([self.x[i][l].data_ptr() for i in range(n_steps) for l in range(len(self.table))])
        yp = B.ptr_array([t.data_ptr() for t in self.y])
        return xp, yp

    def run(self, n_steps=None, stream=None):
        n_steps = len(self.x) if n_steps is None else n_steps
        xp, yp = self.ptrs(n_steps)
        B.dp_plan_run(self.plan, self.kept[:n_steps], 0, xp, yp, self.workspace, self.status,
                      flags=B.DP_PLAN_SAME_Y, stream=stream)

    def capture(self, n_steps=None):
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.run(n_steps)  # warm-up outside capture (lazy module loading, attribute setting)
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            self.run(n_steps)
        return g

    def close(self):
        if self.plan is not None:
            B.dp_plan_destroy(self.plan)
            self.plan = None
