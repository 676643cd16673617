"""The seeded input generator: statistics and structure of the stand-in workloads."""
import numpy as np

from paper_2511_11446_b200 import synth


def test_standard_normal_moments_and_determinism():
    z = synth.std_normal(synth.stream_key(1, synth.KIND_ACT, 2, 3), 0, 1 << 18)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01 and np.abs(z).max() < 4.9
    z2 = synth.std_normal(synth.stream_key(1, synth.KIND_ACT, 2, 3), 1000, 50)
    assert np.array_equal(z2, z[1000:1050])           # counter-based: any slice regenerates
    assert not np.array_equal(z[:50], synth.std_normal(synth.stream_key(1, synth.KIND_ACT, 2, 4), 0, 50))


def test_activation_outliers_rows_and_weights():
    x = synth.activations(5, 1, 2, 32, 1152, 1.0, n_out=12)
    xf = synth.bf16_bits_to_f32(x)
    col = np.abs(xf).mean(axis=0)
    assert (col > 8).sum() == 12                       # 1 % of channels scaled x20
    rows = synth.activations(5, 1, 2, 32, 1152, 1.0, n_out=12, rows=[3, 17])
    assert np.array_equal(rows, x[[3, 17]])
    for bits in (3, 4, 8):
        w, s_w = synth.weights(5, 0, 16, 1152, bits)
        qmax = (1 << (bits - 1)) - 1
        assert w.min() >= -qmax and w.max() <= qmax and np.all(np.abs(w).max(axis=1) == qmax)
        assert np.all(s_w > 0) and abs(np.median(s_w) * qmax / 0.02 - 3.3) < 0.6


def test_plan_schedule_and_layer_table():
    plan = synth.bit_plan(7, 140)
    assert set(plan) == {3, 4, 8} and plan == synth.bit_plan(7, 140)
    kept = synth.kept_timesteps(7, 50, 25, 0.2)
    assert len(kept) == 25 and kept == sorted(kept) and set(range(40, 50)) <= set(kept)
    L = synth.dit_layers(8, 256)
    assert len(L) == 140 and L[0][1:] == (2048, 1152, 3456) and L[4][1:] == (8, 1152, 6912)
    assert synth.gelu_activations(1, 0, 0, 4, 128).shape == (4, 128)
