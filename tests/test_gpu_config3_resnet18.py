"""GPU parity on the ResNet-18 sweep (batch 256, 224x224): every distinct layer shape runs 100
iterations of the fused hot path with a fresh heavy-tailed gradient per iteration whose scale
follows a seeded log-normal random walk (sigma 0.05); the interval state is carried.

Checked against the oracle: at checkpoint iterations the statistics, every gradient code and
sampled int32 accumulators / fp32 outputs at full size; between checkpoints the clipping-factor
trajectory (the oracle's update rule fed with the clip-out counts, which are themselves verified
exactly at the checkpoints and, for the smaller layers, at every iteration).
"""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, shapes, synth
from test_gpu_hot_path import Layer

pytestmark = pytest.mark.gpu

ITERATIONS = 100
SMALL = 26_000_000          # layers up to this many gradient elements are checked at every iteration


@pytest.mark.parametrize("name", list(shapes.CONFIG3))
def test_resnet18_layer_over_100_iterations(name):
    shape, _count = shapes.CONFIG3[name]
    seed = 300 + list(shapes.CONFIG3).index(name)
    layer = Layer(shape, bits=4, seed=seed, gamma=1.0)
    n = layer.n
    walk = synth.lognormal_walk(ITERATIONS, 0.05, seed)
    every = n <= SMALL
    checkpoints = {0, 1, 49, 99} if every else {0, 99}
    gamma = np.float32(1.0)
    for t in range(ITERATIONS):
        dY = synth.laplace_outliers_torch(n, 1e-4 * float(walk[t]), seed=seed, stream=t)
        layer.step(dY)
        stats = lbt.read_stats(layer.stats)
        state = lbt.read_state(layer.st)
        assert state.dev_status == 0 and state.iter == t + 1 and stats.n == n and stats.n_nonfinite == 0
        if t in checkpoints:
            g = dY.cpu().numpy()
            assert layer.gamma == gamma
            rq = layer.check_quantizer(g)          # g_max, n_out, scale, all codes, gamma, iter
            layer.check_contractions(rq, samples=400, seed=t)
        else:
            if every and t % 10 == 5:
                g = dY.cpu().numpy()
                gm, _ = ref.grad_stats(g)
                assert np.float32(stats.g_max) == gm
                assert stats.n_out == ref.clip_count(g, gamma * gm)
            layer.gamma = ref.update_interval(gamma, 1e-3, 1e-3, 1e-3, 1.0, 4, n, stats.n_out)
            layer.it = t + 1
            assert np.float32(state.gamma) == layer.gamma
        gamma = layer.gamma
        del dY
    assert gamma < np.float32(1.0)      # the factor moved away from the min-max baseline
