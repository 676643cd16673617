"""The CUDA input generator reproduces the numpy generator bit for bit."""
import numpy as np
import pytest
import torch

from paper_2511_11446_b200 import synth, synth_cuda
from gpu_util import bf16_to_np

pytestmark = pytest.mark.gpu


def test_activations_identical():
    for (M, K, sig, n_out) in [(64, 1152, 1.0, 12), (9, 4608, 2.34, 46), (300, 128, 0.5, 0)]:
        a = synth.activations(11, 4, 7, M, K, sig, n_out)
        b = bf16_to_np(synth_cuda.activations(11, 4, 7, M, K, sig, n_out))
        assert np.array_equal(a, b)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_weights_identical(bits):
    w, s = synth.weights(11, 2, 96, 1152, bits)
    wg, sg = synth_cuda.weights(11, 2, 96, 1152, bits)
    assert np.array_equal(w, wg.cpu().numpy())
    assert np.array_equal(s.view(np.uint32), sg.cpu().numpy().view(np.uint32))
