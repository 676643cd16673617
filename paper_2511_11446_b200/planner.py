"""Phase A of Algorithm 2 fed by this library's own measured latencies.

`latency_table` times every distinct (layer shape, bit option) of a stack with dp_layer_latency_us
(the whole quantized linear as dp_wq_linear runs it: the c_lat(l, b) input of the algorithm, which the
paper measures with its own integer kernels); `joint_plan` assembles the algorithm's inputs (per-layer
options with measured latency and packed-weight bytes, sensitivities, per-step drift and cost, budgets)
and calls dp_plan_phase_a. Sensitivities and drifts come from the caller: the paper derives them from
its checkpoints and calibration data, which this repository does not have. Bookkeeping only: the
planning arithmetic is in the library.
"""
from __future__ import annotations

from . import binding as B
from .workloads import DevWeights


def latency_table(table, bit_options=(8, 4, 3), seed=1, reps=20):
    """{(M, K, N, bits): microseconds} for the distinct shapes of `table` = [(name, M, K, N)]."""
    out = {}
    for (_, M, K, N) in table:
        for b in bit_options:
            if (M, K, N, b) not in out:
                W = DevWeights(seed, 0, N, K, b)
                out[(M, K, N, b)] = B.dp_layer_latency_us(W.w, M, 0, reps)
    return out


def joint_plan(table, lat, sens, drift, step_overhead_us, B_lat, B_mem, rho=0.2, eps=1e-6, bit_options=(8, 4, 3)):
    """Runs Phase A for the stack `table` with the latency table `lat`.

    One additive latency as in the listing: c_lat(l, b) is the layer's measured time summed over all
    T steps and c_step(t) the bit-plan-independent remainder of a step (`step_overhead_us`), so that
    C_lat starts as the full-precision-plan run time; dropping a step also removes that step's share
    of the current layer times, which the listing's static c_step cannot express, so the returned
    C_lat is an upper bound once steps are dropped (the caller re-times the final plan).
    Returns (bits per layer, kept timesteps ascending, (C_lat, C_mem), feasible)."""
    T = len(drift)
    options = [[(b, T * lat[(M, K, N, b)], N * K * b / 8 + 6 * N) for b in bit_options] for (_, M, K, N) in table]
    plan, kept, totals, ok = B.dp_plan_phase_a(drift, [step_overhead_us] * T, options, sens, B_lat, B_mem, rho, eps)
    return plan, [t for t in range(T) if kept[t]], totals, ok
