"""The bounded device waits, made to run out once (no fault, no hang: a pipeline stage that nothing
fills). The kernel must return by itself, report DP_ERR_TIMEOUT in the caller's status word and
leave the context usable: the same call made again right after is bit-exact against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2511_11446_b200 import binding as B, synth
from gpu_util import DevLayer, run_linear
from helpers import bf16_ulp_dist

pytestmark = pytest.mark.gpu


def test_wait_that_nothing_satisfies_ends_with_timeout_status_and_next_call_is_exact():
    seed, M, K, N, bits = synth.BASE_SEED + 11, 128, 512, 256, 8
    flags = (B.DP_FLAG_FORCE_MMA | B.DP_FLAG_NO_CTA_PAIR | B.DP_FLAG_NO_WEIGHT_STATIONARY |
             B.DP_FLAG_TILE_N(128))               # single-CTA kernel, two CTAs of one tile each
    x = synth.activations(seed, 0, 0, M, K, 1.0, n_out=4)
    w, s_w = synth.weights(seed, 0, N, K, bits)
    b = synth.bias(seed, 0, N)
    L = DevLayer(w, s_w, b, bits)
    B.dp_debug_skip_stage_load(1)                 # k-block 1 of each CTA's first tile gets no loads
    out = run_linear(L, x, flags=flags, taps=False)
    assert out["status"] == B.DP_ERR_TIMEOUT
    # the hook cleared itself with that launch; the context is intact
    out = run_linear(L, x, flags=flags, taps=True)
    assert out["status"] == B.DP_OK
    y, q, s_a, acc = oracle.wq_linear(x, oracle.pack(w, bits), s_w, b, bits, taps=True)
    assert np.array_equal(out["q"], q) and np.array_equal(out["s_a"].view(np.uint32), s_a.view(np.uint32))
    assert np.array_equal(out["acc"], acc)
    assert bf16_ulp_dist(out["y"], y).max() <= 1
    # clearing without a launch
    B.dp_debug_skip_stage_load(2)
    B.dp_debug_skip_stage_load(-1)
    assert run_linear(L, x, flags=flags, taps=False)["status"] == B.DP_OK
