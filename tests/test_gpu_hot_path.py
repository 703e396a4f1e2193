"""GPU parity of the fused hot path (`lbt_qconv_backward`) on the benchmark configurations.

Small configurations are compared element by element; the larger ones on all codes / statistics and
on sampled accumulators the oracle computes one by one.
"""
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, shapes, synth
from tests.guard import Guard

pytestmark = pytest.mark.gpu

S_W, S_X = 0.01, 0.05
THREADS = min(16, os.cpu_count() or 1)


def stratified_indices(rows, cols, rng, block=32, edge_cap=65536):
    """Flat indices into a [rows, cols] matrix: one uniformly random element of every block x block
    cell, every element of the first and last row, and the first and last column (a random subset of
    at most `edge_cap` rows of them when the matrix is taller than that)."""
    rb, cb = (rows + block - 1) // block, (cols + block - 1) // block
    r0 = np.repeat(np.arange(rb, dtype=np.int64) * block, cb)
    c0 = np.tile(np.arange(cb, dtype=np.int64) * block, rb)
    r = r0 + rng.integers(0, np.minimum(block, rows - r0))
    c = c0 + rng.integers(0, np.minimum(block, cols - c0))
    parts = [r * cols + c, np.arange(cols, dtype=np.int64), (rows - 1) * cols + np.arange(cols, dtype=np.int64)]
    edge_rows = np.arange(rows, dtype=np.int64) if rows <= edge_cap else rng.integers(0, rows, edge_cap)
    parts += [edge_rows * cols, edge_rows * cols + (cols - 1)]
    return np.concatenate(parts)


class Layer:
    def __init__(self, shape, bits=4, seed=0, gamma=1.0, want_acc=True):
        self.shape, self.bits, self.seed = shape, bits, seed
        self.d, self.desc = ref.ConvShape(**shape), lbt.ConvDesc(**shape)
        d = self.d
        self.n = d.N * d.P * d.Q * d.K
        self.raw_w = synth.code_bytes_torch(d.K * d.R * d.S * d.C // 2 + 1, seed, 1)[: (d.K * d.R * d.S * d.C + 1) // 2]
        self.raw_x = synth.code_bytes_torch((d.N * d.H * d.W * d.C + 1) // 2, seed, 2)
        self.st = lbt.new_state(gamma=gamma, bits=bits, rounding=lbt.ROUND_STOCHASTIC, seed=seed)
        self.stats = lbt.new_stats()
        self.sc = torch.tensor([S_W, S_X], device="cuda")
        self.guard = Guard()          # every output and the workspace are followed by a canary
        self.q_dY = self.guard.alloc((self.n + 1) // 2 if bits <= 4 else self.n, torch.uint8)
        self.dX = self.guard.alloc((d.N, d.H, d.W, d.C), torch.float32)
        self.dW = self.guard.alloc((d.K, d.R, d.S, d.C), torch.float32)
        self.accX = self.guard.alloc(self.dX.shape, torch.int32) if want_acc else None
        self.accW = self.guard.alloc(self.dW.shape, torch.int32) if want_acc else None
        self.ws = self.guard.alloc(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, self.desc), torch.uint8)
        self.gamma = np.float32(gamma)
        self.it = 0
        self._cw = self._cx = None

    def step(self, dY):
        lbt.qconv_backward(self.desc, dY, self.raw_w, self.raw_x, self.sc.data_ptr(), self.sc.data_ptr() + 4,
                           self.st, self.stats, self.q_dY, self.dX, self.dW, self.accX, self.accW, self.bits, self.ws)
        torch.cuda.synchronize()

    def oracle_quantizer(self, g):
        gm, bad = ref.grad_stats(g)
        rq = ref.quantize_grad(g, self.gamma, gm, self.bits, 1, self.seed, self.it, bad)
        new_gamma = ref.update_interval(self.gamma, 1e-3, 1e-3, 1e-3, 1.0, self.bits, g.size, rq.n_out, bad)
        return gm, rq, new_gamma

    def check_quantizer(self, g):
        gm, rq, new_gamma = self.oracle_quantizer(g)
        s = lbt.read_stats(self.stats)
        assert np.float32(s.g_max) == gm and s.n_out == rq.n_out and np.float32(s.scale) == rq.scale
        assert np.array_equal(self.q_dY.cpu().numpy(), ref.pack(rq.codes, self.bits))
        state = lbt.read_state(self.st)
        assert np.float32(state.gamma) == new_gamma and state.dev_status == 0 and state.iter == self.it + 1
        self.gamma, self.it = new_gamma, self.it + 1
        return rq

    def operand_codes(self):
        if self._cw is None:
            d = self.d
            self._cw = ref.unpack4(self.raw_w.cpu().numpy(), d.K * d.R * d.S * d.C, True)
            self._cx = ref.unpack4(self.raw_x.cpu().numpy(), d.N * d.H * d.W * d.C, False)
        return self._cw, self._cx

    def check_contractions(self, rq, samples=None, seed=0, strata=True):
        """Accumulators and fp32 outputs against the oracle: every output when `samples` is None, else
        `samples` uniformly random outputs plus (strata) one random output in every 32 x 32 block of the
        output matrix ([pixels, C] for dX, [K, R S C] for dW) and its first / last rows and columns, so
        that every tile of the persistent kernels, and every epilogue block inside it, is looked at."""
        self.guard.check()
        cw, cx = self.operand_codes()
        cy = rq.codes.astype(np.int16)
        for kind, other, acc, out, s_o in (("dgrad", cw, self.accX, self.dX, S_W), ("wgrad", cx, self.accW, self.dW, S_X)):
            total = out.numel()
            if samples is None or samples >= total:
                want = ref.conv_backward(kind, self.d, cy, other, threads=THREADS).ravel()
                got_acc, got = acc.cpu().numpy().ravel(), out.cpu().numpy().ravel()
            else:
                rng = np.random.default_rng(seed)
                idx = rng.integers(0, total, samples)
                if strata:
                    rows = out.shape[0] if kind == "wgrad" else total // out.shape[-1]
                    idx = np.concatenate([idx, stratified_indices(rows, total // rows, rng)])
                want = ref.conv_backward(kind, self.d, cy, other, idx=idx, threads=THREADS)
                t = torch.from_numpy(idx).cuda()
                got_acc, got = acc.view(-1)[t].cpu().numpy(), out.view(-1)[t].cpu().numpy()
            assert np.array_equal(got_acc, want.astype(np.int32)), kind
            f, over = ref.epilogue(want, rq.scale, s_o)
            assert over == 0
            tol = 1e-6 * np.abs(f) + 1e-6 * float(np.float32(rq.scale) * np.float32(s_o))
            assert np.all(np.abs(got - f) <= tol), kind


def test_config0_single_linear_layer():
    layer = Layer(shapes.CONFIG0["linear_128x256x256"], seed=0)
    g = synth.laplace_outliers(128 * 256, 1e-3, seed=0)
    layer.step(torch.from_numpy(g).cuda())
    layer.check_contractions(layer.check_quantizer(g))


def test_config1_ten_drifting_steps():
    layer = Layer(shapes.CONFIG1["resnet20_3x3_16"], seed=1)
    for t in range(10):
        g = synth.laplace_outliers(layer.n, 1e-4 * 0.9 ** t, seed=1, stream=t)
        layer.step(torch.from_numpy(g).cuda())
        rq = layer.check_quantizer(g)
        if t in (0, 9):
            layer.check_contractions(rq, samples=20000, seed=t)


@pytest.mark.parametrize("name", list(shapes.CONFIG2))
def test_config2_resnet50_layers(name):
    layer = Layer(shapes.CONFIG2[name], seed=2, gamma=0.8)
    dY = synth.student_t3_torch(layer.n, 1e-4, seed=2)
    layer.step(dY)
    rq = layer.check_quantizer(dY.cpu().numpy())
    layer.check_contractions(rq, samples=3000)


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_config4_edsr_layer_bit_widths(bits):
    layer = Layer(shapes.CONFIG4["edsr_3x3_64"], bits=bits, seed=4, gamma=0.6)
    dY = synth.laplace_outliers_torch(layer.n, 1e-3, seed=4)
    layer.step(dY)
    rq = layer.check_quantizer(dY.cpu().numpy())
    layer.check_contractions(rq, samples=3000)


def test_nonfinite_gradient_is_reported_and_outputs_stay_defined():
    layer = Layer(shapes.conv(2, 16, 8, 8, 16, 3, 3, 1, 1), seed=5, gamma=0.5)
    g = synth.laplace_outliers(layer.n, 1e-3, seed=5)
    g[7] = np.nan
    layer.step(torch.from_numpy(g).cuda())
    state = lbt.read_state(layer.st)
    assert state.dev_status == lbt.ERR_NONFINITE and np.float32(state.gamma) == np.float32(0.5)
    assert not layer.q_dY.any() and not layer.accX.any() and not layer.accW.any()
    assert not layer.dX.any() and not layer.dW.any()


@pytest.mark.parametrize("n_elems_shape", [shapes.conv(2, 16, 8, 8, 16, 3, 3, 1, 1), shapes.conv(64, 256, 1, 1, 512, 1, 1, 1, 0)],
                         ids=["conv3x3", "linear"])
@pytest.mark.parametrize("state_bits,call_bits", [(8, 4), (4, 8), (6, 4)])
def test_bit_width_that_differs_from_the_state_is_reported(n_elems_shape, state_bits, call_bits):
    """bits_g sizes the code buffer and the integer pipeline on the host; a device state with another width
    must not be quantized into it: status LBT_ERR_BITS_MISMATCH, zero codes and outputs, gamma untouched,
    and nothing written past the (smaller) code buffer."""
    layer = Layer(n_elems_shape, bits=call_bits, seed=6, gamma=0.5)
    layer.st = lbt.new_state(gamma=0.5, bits=state_bits, rounding=lbt.ROUND_STOCHASTIC, seed=6)
    g = synth.laplace_outliers(layer.n, 1e-3, seed=6)
    layer.step(torch.from_numpy(g).cuda())
    layer.guard.check()
    state = lbt.read_state(layer.st)
    assert state.dev_status == lbt.ERR_BITS_MISMATCH and np.float32(state.gamma) == np.float32(0.5)
    assert state.iter == 1
    assert lbt.status_string(state.dev_status) == "LBT_ERR_BITS_MISMATCH"
    assert not layer.q_dY.any() and not layer.accX.any() and not layer.accW.any()
    assert not layer.dX.any() and not layer.dW.any()
