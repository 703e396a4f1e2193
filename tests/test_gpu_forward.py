"""GPU parity, forward side: the weight / activation quantizers (Eq. 1-4) and the integer forward
product versus the CPU oracle.  Codes, scales and int32 accumulators bit for bit; fp32 outputs
within 1e-6 relative."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, shapes, synth
from tests.guard import Guard
from tests.test_gpu_contractions import CONVS, LINEAR, PERSISTENT_CONVS, THREADS, _check_out, _codes_for, _status_ok

pytestmark = pytest.mark.gpu

S_X, S_W = 0.05, 0.01


def _quantize(kind, x_host, c, bits):
    x = torch.from_numpy(x_host).cuda()
    n = x.numel()
    q = torch.full(((n + 1) // 2 if bits <= 4 else n,), 0xA5, dtype=torch.uint8, device="cuda")
    io = torch.tensor([c, -1.0], dtype=torch.float32, device="cuda")      # clip in, scale out
    fn = lbt.quantize_weight if kind == "weight" else lbt.quantize_act
    fn(x, io.data_ptr(), bits, q, io.data_ptr() + 4)
    torch.cuda.synchronize()
    raw = q.cpu().numpy()
    if bits <= 4:
        codes = ref.unpack4(raw, n, kind == "weight")
    else:
        codes = raw.view(np.int8).astype(np.int16) if kind == "weight" else raw.astype(np.int16)
    return codes, raw, np.float32(io[1].item())


def _inputs(n, seed):
    x = synth.laplace_outliers(n, 0.05, seed)
    x[::97] = 0.0
    if n > 40:
        x[5], x[6], x[7], x[8] = np.inf, -np.inf, np.nan, -0.0
        x[9], x[10] = 1e-45, -1e-30                                     # subnormal, tiny
    return x


def _oracle(kind):
    return ref.quantize_weight if kind == "weight" else ref.quantize_act


@pytest.mark.parametrize("kind", ["weight", "act"])
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 8])
@pytest.mark.parametrize("n", [1, 7, 8, 9, 4097, 300_003])
def test_forward_quantizer_codes_and_scale(kind, bits, n):
    x = _inputs(n, 3 * bits + n % 5)
    c = np.float32(0.21)
    want_codes, want_s = _oracle(kind)(x, c, bits)
    codes, raw, s = _quantize(kind, x, c, bits)
    assert s == want_s
    assert np.array_equal(codes, want_codes.astype(np.int16))
    if bits <= 4 and n % 2:
        assert raw[-1] >> 4 == 0                                          # odd tail padded with 0
    if kind == "weight":
        assert np.array_equal(raw, ref.pack(want_codes.astype(np.int8), bits))


@pytest.mark.parametrize("kind", ["weight", "act"])
@pytest.mark.parametrize("c", [0.0, -1.0, float("nan"), float("inf"), 1e-30, 3e25, 1e-22])
def test_forward_quantizer_extreme_clipping_values(kind, c):
    """Degenerate c gives zero codes and scale 0; very small / very large c leaves the range of the
    fast division and takes the division routine: same codes as the oracle either way."""
    x = _inputs(5000, 11) * np.float32(c * 60 if np.isfinite(c) and c > 0 else 1.0)   # a few per cent clipped
    want_codes, want_s = _oracle(kind)(x, c, 4)
    codes, _, s = _quantize(kind, x, c, 4)
    assert s == want_s
    assert np.array_equal(codes, want_codes.astype(np.int16))


def test_forward_quantizer_large_tensor_spans_the_whole_grid():
    n = 12_845_056 + 3                                                   # more groups than threads in the grid
    x = synth.laplace_outliers(n, 0.02, 5)
    for kind, bits in (("weight", 4), ("act", 4), ("act", 8)):
        want_codes, want_s = _oracle(kind)(x, 0.07, bits)
        codes, _, s = _quantize(kind, x, 0.07, bits)
        assert s == want_s and np.array_equal(codes, want_codes.astype(np.int16))


def test_forward_quantizer_rejections():
    L = lbt.lib()
    buf = torch.zeros(64, device="cuda")
    p = buf.data_ptr()
    assert L.lbt_quantize_weight(p, 8, p, 9, p, p, 0) == lbt.ERR_UNSUPPORTED_BITS
    assert L.lbt_quantize_act(p, 8, p, 1, p, p, 0) == lbt.ERR_UNSUPPORTED_BITS
    assert L.lbt_quantize_weight(p, 8, None, 4, p, p, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_quantize_act(None, 8, p, 4, p, p, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_quantize_act(p + 4, 8, p, 4, p, p, 0) == lbt.ERR_ALIGNMENT


# ------------------------------------------------------------------------------ forward product
def _scales():
    return torch.tensor([S_X, S_W], dtype=torch.float32, device="cuda")


# the last two: 128 CTA-pair tiles on 74 pairs; 200 single-CTA tiles on 148 SMs (several tiles per CTA)
@pytest.mark.parametrize("M,O,I", LINEAR + [(300, 520, 200), (513, 256, 384), (4096, 2048, 256), (25600, 96, 64),
                                          (20224, 256, 200), (24064, 256, 72)],   # 5 left-over tiles cut into 4 column slices; 20 left over: not cut
                         ids=lambda v: str(v))
@pytest.mark.parametrize("bits_x", [4, 8])
def test_linear_forward(M, O, I, bits_x):
    q_X, c_X = _codes_for(M * I, bits_x, False, 4, 2)
    q_W, c_W = _codes_for(O * I, 4, True, 4, 1)
    sc = _scales()
    guard = Guard()
    ws = guard.alloc(lbt.workspace_bytes(lbt.OP_GEMM_FORWARD, lbt.GemmDesc(M, O, I)), torch.uint8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = guard.alloc((M, O), torch.float32, float("nan"))
    acc = guard.alloc((M, O), torch.int32, -77)
    lbt.qgemm_forward(q_X, q_W, sc.data_ptr(), sc.data_ptr() + 4, Y, acc, M, O, I, bits_x, 4, ws, status)
    _status_ok(status)
    guard.check()
    _check_out(Y, acc, ref.gemm_forward(c_X, c_W, M, O, I, threads=THREADS), S_X, S_W)


def _conv_forward(shape, seed):
    d = ref.ConvShape(**shape)
    desc = lbt.ConvDesc(**shape)
    q_X, c_X = _codes_for(d.N * d.H * d.W * d.C, 4, False, seed, 2)
    q_W, c_W = _codes_for(d.K * d.R * d.S * d.C, 4, True, seed, 1)
    sc = _scales()
    guard = Guard()
    ws = guard.alloc(lbt.workspace_bytes(lbt.OP_CONV_FORWARD, desc), torch.uint8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = guard.alloc((d.N, d.P, d.Q, d.K), torch.float32, float("nan"))
    acc = guard.alloc(Y.shape, torch.int32, -77)
    lbt.qconv_forward(desc, q_X, q_W, sc.data_ptr(), sc.data_ptr() + 4, Y, acc, 4, 4, ws, status)
    _status_ok(status)
    guard.check()
    return d, c_X, c_W, Y, acc


@pytest.mark.parametrize("shape", CONVS + PERSISTENT_CONVS,
                         ids=lambda s: "N{N}C{C}H{H}K{K}R{R}s{stride}p{pad}".format(**s))
def test_convolution_forward(shape):
    d, c_X, c_W, Y, acc = _conv_forward(shape, 5)
    _check_out(Y, acc, ref.conv_forward(d, c_X, c_W, threads=THREADS), S_X, S_W)


_FULL_SIZE = {
    "resnet50_3x3_256_256": shapes.CONFIG2["resnet50_3x3_256_256"],      # CTA-pair tiles, row window + B ring
    "resnet50_1x1_256_1024": shapes.CONFIG2["resnet50_1x1_256_1024"],    # CTA-pair tiles, one tap
    "resnet18_layer1": shapes.CONFIG3["layer1"][0],                      # window + resident filter, 2 window buffers
    "resnet18_layer2": shapes.CONFIG3["layer2"][0],                      # resident filter, 1 window buffer
    "resnet18_layer2.0.conv1": shapes.CONFIG3["layer2.0.conv1"][0],      # stride 2: one box per tap
    "edsr_3x3_64": shapes.CONFIG4["edsr_3x3_64"],                        # wide images: 3-box window
    "resnet20_3x3_16": list(shapes.CONFIG1.values())[0],                 # 16 channels
}


@pytest.mark.parametrize("name", list(_FULL_SIZE))
def test_forward_on_full_size_layers_sampled(name):
    """Full-size layers (every tile shape and operand-feed mode of the forward product): 4000 sampled outputs."""
    d, c_X, c_W, Y, acc = _conv_forward(_FULL_SIZE[name], 6)
    total = Y.numel()
    idx = np.unique(np.concatenate([np.random.default_rng(1).integers(0, total, 4000),
                                    [0, total - 1, d.K - 1, d.K, total - d.K]]))
    want = ref.conv_forward(d, c_X, c_W, idx=idx, threads=8)
    assert np.array_equal(acc.cpu().numpy().ravel()[idx], want.astype(np.int32))
    out, over = ref.epilogue(want, S_X, S_W)
    assert over == 0 and np.allclose(Y.cpu().numpy().ravel()[idx], out, rtol=1e-6, atol=0)
    assert not torch.isnan(Y).any()


def test_quantize_then_forward_end_to_end():
    """Weights and activations quantized on the device feed the forward product directly."""
    M, O, I = 384, 272, 200
    x = np.abs(synth.laplace_outliers(M * I, 0.5, 8))
    w = synth.laplace_outliers(O * I, 0.05, 9)
    io = torch.tensor([1.7, 0.16, 0.0, 0.0], dtype=torch.float32, device="cuda")   # c_x, c_w, s_x, s_w
    q_X = torch.empty(M * I // 2, dtype=torch.uint8, device="cuda")
    q_W = torch.empty(O * I // 2, dtype=torch.uint8, device="cuda")
    lbt.quantize_act(torch.from_numpy(x).cuda(), io.data_ptr(), 4, q_X, io.data_ptr() + 8)
    lbt.quantize_weight(torch.from_numpy(w).cuda(), io.data_ptr() + 4, 4, q_W, io.data_ptr() + 12)
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_GEMM_FORWARD, lbt.GemmDesc(M, O, I)), dtype=torch.uint8, device="cuda")
    Y = torch.empty(M, O, device="cuda")
    acc = torch.empty(M, O, dtype=torch.int32, device="cuda")
    lbt.qgemm_forward(q_X, q_W, io.data_ptr() + 8, io.data_ptr() + 12, Y, acc, M, O, I, 4, 4, ws)
    torch.cuda.synchronize()
    cx, sx = ref.quantize_act(x, 1.7, 4)
    cw, sw = ref.quantize_weight(w, 0.16, 4)
    _check_out(Y, acc, ref.gemm_forward(cx, cw, M, O, I, threads=8), sx, sw)


def test_forward_host_side_rejections():
    L = lbt.lib()
    sc = _scales()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    out = torch.zeros(1 << 12, device="cuda")
    p, o = buf.data_ptr(), out.data_ptr()
    need = lbt.workspace_bytes(lbt.OP_GEMM_FORWARD, lbt.GemmDesc(8, 8, 8))
    assert need > 0
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    call = lambda M, O, I, bx, bw, wsp, wsb, y=o: L.lbt_qgemm_forward(p, p, sc.data_ptr(), sc.data_ptr() + 4, y, None,
                                                                      M, O, I, bx, bw, None, wsp, wsb, 0)
    assert call(8, 8, 8, 4, 4, ws.data_ptr(), need - 1) == lbt.ERR_WORKSPACE
    assert call(8, 8, 8, 4, 9, ws.data_ptr(), need) == lbt.ERR_UNSUPPORTED_BITS
    assert call(8, 8, 0, 4, 4, ws.data_ptr(), need) == lbt.ERR_INVALID_ARG
    assert call(8, 8, 8, 4, 4, ws.data_ptr(), need, None) == lbt.ERR_INVALID_ARG
    assert call(8, 8, 1 << 17, 8, 8, ws.data_ptr(), 1 << 40) == lbt.ERR_ACC_RANGE
    bad = lbt.ConvDesc(N=1, C=1, H=8, W=8, K=1, R=3, S=3, stride=3, pad=1)
    assert lbt.workspace_bytes(lbt.OP_CONV_FORWARD, bad) == 0
    assert L.lbt_qconv_forward(ctypes.addressof(bad), p, p, sc.data_ptr(), sc.data_ptr() + 4, o, None, 4, 4, None,
                               ws.data_ptr(), need, 0) == lbt.ERR_UNSUPPORTED
