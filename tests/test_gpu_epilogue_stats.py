"""The next layer's statistics out of the dgrad epilogue (`lbt_qconv_backward_ex`): the abs-max, the
element count and the non-finite count of dX must be what the statistics pass would compute on dX (the
oracle's `grad_stats` of the oracle's dX), bit for bit; and a layer that trusts them (dy_stats_ready)
must produce the oracle's codes without running its own abs-max pass."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, shapes, synth
from tests.guard import Guard

pytestmark = pytest.mark.gpu


class _Layer:
    def __init__(self, shape, bits=4, seed=0, gamma=0.8, s_w=0.01, s_x=0.05, want_acc=False):
        self.shape, self.bits, self.seed, self.gamma, self.s_w, self.s_x = shape, bits, seed, np.float32(gamma), s_w, s_x
        self.d, self.desc = ref.ConvShape(**shape), lbt.ConvDesc(**shape)
        d = self.d
        self.n = d.N * d.P * d.Q * d.K
        self.raw_w = synth.code_bytes((d.K * d.R * d.S * d.C + 1) // 2, seed, 1)
        self.raw_x = synth.code_bytes((d.N * d.H * d.W * d.C + 1) // 2, seed, 2)
        self.q_W, self.q_X = torch.from_numpy(self.raw_w).cuda(), torch.from_numpy(self.raw_x).cuda()
        self.st = lbt.new_state(gamma=gamma, bits=bits, rounding=lbt.ROUND_STOCHASTIC, seed=seed)
        self.stats, self.dx_stats = lbt.new_stats(), lbt.new_stats()
        self.dx_stats.fill_(0xEE)                       # the call must clear it
        self.sc = torch.tensor([s_w, s_x], device="cuda")
        g = self.guard = Guard()
        self.q_dY = g.alloc((self.n + 1) // 2 if bits <= 4 else self.n, torch.uint8)
        self.dX = g.alloc((d.N, d.H, d.W, d.C), torch.float32, float("nan"))
        self.dW = g.alloc((d.K, d.R, d.S, d.C), torch.float32, float("nan"))
        self.accX = g.alloc(self.dX.shape, torch.int32, -77) if want_acc else None
        self.ws = g.alloc(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, self.desc), torch.uint8)

    def run(self, dY, stats_ready=False, want_dx_stats=True):
        lbt.qconv_backward_ex(self.desc, dY, self.q_W, self.q_X, self.sc.data_ptr(), self.sc.data_ptr() + 4, self.st,
                              self.stats, self.q_dY, self.dX, self.dW, self.accX, None, self.bits, self.ws,
                              dy_stats_ready=stats_ready, dx_stats=self.dx_stats if want_dx_stats else None)
        torch.cuda.synchronize()
        self.guard.check()
        assert lbt.read_state(self.st).dev_status == 0

    def oracle_dx(self, g):
        """The oracle's quantization of g and the dX it leads to (fp32)."""
        gm, bad = ref.grad_stats(g)
        rq = ref.quantize_grad(g, self.gamma, gm, self.bits, 1, self.seed, 0, bad)
        cw = ref.unpack4(self.raw_w, self.d.K * self.d.R * self.d.S * self.d.C, True)
        acc = ref.conv_backward("dgrad", self.d, rq.codes, cw, threads=8)
        dx, over = ref.epilogue(acc, rq.scale, self.s_w)
        assert over == 0
        return rq, dx


SHAPES = {
    "linear_tma_store": shapes.linear(384, 256, 512),                         # flat output: TMA-store epilogue, CTA pairs
    "linear_narrow": shapes.linear(300, 72, 40),                              # 40 of 48 padded columns exist: ragged chunk
    "conv3x3_halo": shapes.conv(3, 20, 9, 9, 40, 3, 3, 1, 1),                 # halo rows must not count
    "conv3x3_stride2": shapes.conv(4, 16, 14, 14, 32, 3, 3, 2, 1),            # parity classes, some without taps
    "conv1x1_stride2": shapes.conv(2, 24, 6, 6, 16, 1, 1, 2, 0),              # three of four classes are all zeros
    "conv3x3_pairs_window": shapes.conv(8, 256, 14, 14, 144, 3, 3, 1, 1),     # CTA pairs, row window
    "conv3x3_64_resident": shapes.conv(4, 64, 16, 16, 64, 3, 3, 1, 1),        # single CTA, resident filter, 8 epilogue warps
    "linear_left_over_slices": shapes.linear(20224, 96, 256),                 # 79 pair tiles: the last 5 cut into 4 column slices
}


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("want_acc", [False, True], ids=["fp32_only", "with_accumulators"])
def test_epilogue_statistics_equal_the_statistics_pass_on_dx(name, want_acc):
    layer = _Layer(SHAPES[name], seed=21, want_acc=want_acc)
    g = synth.laplace_outliers(layer.n, 1e-3, seed=21)
    layer.run(torch.from_numpy(g).cuda())
    rq, dx = layer.oracle_dx(g)
    assert np.array_equal(layer.dX.cpu().numpy().ravel(), dx.ravel())
    want_gmax, want_bad = ref.grad_stats(dx)
    s = lbt.read_stats(layer.dx_stats)
    assert np.float32(s.g_max) == want_gmax and want_gmax > 0
    assert (s.n, s.n_nonfinite, s.n_out, s.reserved) == (dx.size, want_bad, 0, 0) and want_bad == 0
    assert s.c == 0.0 and s.scale == 0.0


def test_a_scale_that_overflows_is_counted_like_the_statistics_pass_would():
    """With a weight scale so large that the products of the larger accumulators overflow, the non-finite
    outputs are counted and left out of the abs-max, as lbt_grad_stats does."""
    layer = _Layer(shapes.conv(3, 20, 9, 9, 40, 3, 3, 1, 1), seed=22)
    g = synth.laplace_outliers(layer.n, 1.0, seed=22)
    # pick s_w so that about a tenth of the accumulators overflow: |acc| * s_g * s_w > FLT_MAX
    gm, bad = ref.grad_stats(g)
    rq = ref.quantize_grad(g, layer.gamma, gm, 4, 1, 22, 0, bad)
    cw = ref.unpack4(layer.raw_w, layer.d.K * 9 * layer.d.C, True)
    acc = np.abs(ref.conv_backward("dgrad", layer.d, rq.codes, cw, threads=8))
    layer.s_w = float(np.float32(3.0e38 / (float(rq.scale) * float(np.percentile(acc, 90)))))
    assert np.isfinite(layer.s_w)
    layer.sc = torch.tensor([layer.s_w, 0.05], device="cuda")
    layer.run(torch.from_numpy(g).cuda())
    with np.errstate(over="ignore"):
        _, dx = layer.oracle_dx(g)
        want_gmax, want_bad = ref.grad_stats(dx)
    assert 0 < want_bad < dx.size and np.isfinite(want_gmax)
    s = lbt.read_stats(layer.dx_stats)
    assert np.float32(s.g_max) == want_gmax and s.n_nonfinite == want_bad and s.n == dx.size
    assert np.array_equal(layer.dX.cpu().numpy().ravel().view(np.uint32), dx.ravel().view(np.uint32))


def test_all_zero_gradient_gives_zero_statistics():
    layer = _Layer(SHAPES["conv3x3_halo"], seed=23)
    layer.run(torch.zeros(layer.n, device="cuda"))
    s = lbt.read_stats(layer.dx_stats)
    assert (s.g_max, s.n, s.n_nonfinite) == (0.0, layer.dX.numel(), 0)
    assert not layer.dX.any()


@pytest.mark.parametrize("second,first", [
    (shapes.linear(256, 192, 320), shapes.linear(256, 320, 128)),             # two linear layers, nothing between
    (shapes.conv(4, 32, 12, 12, 48, 3, 3, 1, 1), shapes.conv(4, 16, 12, 12, 32, 3, 3, 1, 1)),
], ids=["linear_chain", "conv_chain"])
def test_two_layer_chain_without_the_second_abs_max_pass(second, first):
    """Layer 2's backward pass leaves dX and its statistics; layer 1 takes that dX as its gradient with
    dy_stats_ready: codes, scale, clip-out count and gamma equal the oracle's, which runs its own statistics."""
    l2 = _Layer(second, seed=31)
    g2 = synth.laplace_outliers(l2.n, 1e-3, seed=31)
    l2.run(torch.from_numpy(g2).cuda())
    l1 = _Layer(first, seed=32, gamma=0.6)
    assert l1.n == l2.dX.numel()
    l1.stats.copy_(l2.dx_stats)                          # (a training loop would pass the same struct)
    l1.run(l2.dX.view(-1), stats_ready=True, want_dx_stats=False)
    g1 = l2.dX.cpu().numpy().ravel()
    gm, bad = ref.grad_stats(g1)
    rq = ref.quantize_grad(g1, np.float32(0.6), gm, 4, 1, 32, 0, bad)
    s = lbt.read_stats(l1.stats)
    assert np.float32(s.g_max) == gm and s.n == g1.size and s.n_out == rq.n_out and np.float32(s.scale) == rq.scale
    assert np.array_equal(l1.q_dY.cpu().numpy(), ref.pack(rq.codes, 4))
    state = lbt.read_state(l1.st)
    assert np.float32(state.gamma) == ref.update_interval(0.6, 1e-3, 1e-3, 1e-3, 1.0, 4, g1.size, rq.n_out, bad)
    assert state.iter == 1
    cw = ref.unpack4(l1.raw_w, l1.d.K * l1.d.R * l1.d.S * l1.d.C, True)
    want, _ = ref.epilogue(ref.conv_backward("dgrad", l1.d, rq.codes, cw, threads=8), rq.scale, l1.s_w)
    assert np.array_equal(l1.dX.cpu().numpy().ravel(), want.ravel())
    assert bytes(l1.dx_stats.cpu().numpy()) == b"\xee" * 40          # not passed: untouched


def test_argument_checks():
    layer = _Layer(SHAPES["conv3x3_halo"], seed=24)
    L = lbt.lib()
    import ctypes
    dY = torch.zeros(layer.n, device="cuda")
    args = lambda dX, dxs: (ctypes.addressof(layer.desc), dY.data_ptr(), layer.q_W.data_ptr(), layer.q_X.data_ptr(),
                            layer.sc.data_ptr(), layer.sc.data_ptr() + 4, layer.st.data_ptr(), layer.stats.data_ptr(),
                            layer.q_dY.data_ptr(), dX, layer.dW.data_ptr(), None, None, 4, layer.ws.data_ptr(),
                            layer.ws.numel(), 0, dxs, 0)
    assert L.lbt_qconv_backward_ex(*args(None, layer.dx_stats.data_ptr())) == lbt.ERR_INVALID_ARG   # statistics of no dX
    assert L.lbt_qconv_backward_ex(*args(layer.dX.data_ptr(), layer.stats.data_ptr())) == lbt.ERR_INVALID_ARG
    assert L.lbt_qconv_backward_ex(*args(layer.dX.data_ptr(), layer.dx_stats.data_ptr() + 4)) == lbt.ERR_ALIGNMENT
