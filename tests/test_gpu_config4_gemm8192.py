"""GPU parity at the benchmark's full size and launch configuration: linear M = O = I = 8192, gradient
bit-widths 4, 6 and 8, through the fused call `bench.py` times.  All statistics and codes are compared;
accumulators and fp32 outputs on sampled entries the oracle computes one by one."""
import pytest

from paper_2407_12637_b200 import shapes, synth
from test_gpu_hot_path import Layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_square_layer_8192(bits):
    layer = Layer(shapes.CONFIG4["gemm_8192"], bits=bits, seed=40 + bits, gamma=0.9)
    dY = synth.laplace_outliers_torch(layer.n, 1e-3, seed=40 + bits)
    layer.step(dY)
    rq = layer.check_quantizer(dY.cpu().numpy())
    layer.check_contractions(rq, samples=1500, seed=bits)
