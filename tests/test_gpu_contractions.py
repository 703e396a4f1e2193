"""GPU parity: integer backward contractions versus the CPU oracle.

int32 accumulators must match bit for bit; the dequantised fp32 outputs within 1e-6 relative
(they are (float)acc * fl32(s_a * s_b) on both sides, so they in fact agree exactly).
"""
import ctypes
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, synth
from tests.guard import Guard

pytestmark = pytest.mark.gpu

S_G, S_W, S_X = 1.25e-4, 0.01, 0.05
THREADS = min(16, os.cpu_count() or 1)


def _scales():
    return torch.tensor([S_G, S_W, S_X], dtype=torch.float32, device="cuda")


def _sptr(t, i):
    return t.data_ptr() + 4 * i


def _codes_for(nelem, bits, signed, seed, stream):
    """Random stored codes: (device bytes as the library reads them, int16 codes for the oracle)."""
    if bits <= 4:
        raw = synth.code_bytes((nelem + 1) // 2, seed, stream)
        if bits < 4:   # keep each nibble inside the b-bit range (sign-extended within the nibble)
            lo, hi = raw & 0xF, raw >> 4
            m = (1 << bits) - 1
            if signed:
                f = lambda v: (((v & m) ^ (1 << (bits - 1))) - (1 << (bits - 1))) & 0xF
            else:
                f = lambda v: v & m
            raw = (f(lo.astype(np.int32)) | (f(hi.astype(np.int32)) << 4)).astype(np.uint8)
        codes = ref.unpack4(raw, nelem, signed)
    else:
        raw = synth.code_bytes(nelem, seed, stream)
        if bits < 8:
            raw = raw >> (8 - bits) if not signed else \
                ((raw.view(np.int8) >> (8 - bits)).view(np.uint8))
        codes = raw.view(np.int8).astype(np.int16) if signed else raw.astype(np.int16)
    return torch.from_numpy(raw).cuda(), codes


def _check_out(out_gpu, acc_gpu, acc_ref, s_a, s_b):
    acc_ref = np.asarray(acc_ref)
    assert np.array_equal(acc_gpu.cpu().numpy().ravel(), acc_ref.ravel().astype(np.int32))
    want, over = ref.epilogue(acc_ref, s_a, s_b)
    assert over == 0
    got = out_gpu.cpu().numpy().ravel()
    tol = 1e-6 * np.abs(want.ravel()) + 1e-6 * float(np.float32(s_a) * np.float32(s_b))
    assert np.all(np.abs(got - want.ravel()) <= tol)


def _status_ok(status):
    torch.cuda.synchronize()
    assert int(status.item()) == 0, lbt.status_string(int(status.item()))


LINEAR = [(128, 256, 256), (1, 1, 1), (5, 3, 7), (130, 72, 40), (257, 129, 300), (64, 600, 130),
          (1000, 16, 16)]


@pytest.mark.parametrize("M,O,I", LINEAR, ids=lambda v: str(v))
@pytest.mark.parametrize("bits_g", [4, 8])
def test_linear_layer(M, O, I, bits_g):
    q_dY, c_dY = _codes_for(M * O, bits_g, True, 1, 0)
    q_W, c_W = _codes_for(O * I, 4, True, 1, 1)
    q_X, c_X = _codes_for(M * I, 4, False, 1, 2)
    sc = _scales()
    desc = lbt.GemmDesc(M, O, I)
    _linear_backward_exhaustive(M, O, I, bits_g, (q_dY, c_dY), (q_W, c_W), (q_X, c_X))


def _linear_backward_exhaustive(M, O, I, bits_g, dy, w, x, kinds=("dgrad", "wgrad"), threads=1):
    """Both contractions of a linear layer, every accumulator and output against the oracle; outputs and
    workspaces are followed by canaries."""
    (q_dY, c_dY), (q_W, c_W), (q_X, c_X) = dy, w, x
    sc = _scales()
    desc = lbt.GemmDesc(M, O, I)
    guard = Guard()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if "dgrad" in kinds:
        ws = guard.alloc(lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, desc), torch.uint8)
        dX = guard.alloc((M, I), torch.float32, float("nan"))
        accX = guard.alloc((M, I), torch.int32, -77)
        lbt.qgemm_dgrad(q_dY, q_W, _sptr(sc, 0), _sptr(sc, 1), dX, accX, M, O, I, bits_g, 4, ws, status)
        _status_ok(status)
        _check_out(dX, accX, ref.gemm_backward("dgrad", c_dY, c_W, M, O, I, threads=threads), S_G, S_W)
    if "wgrad" in kinds:
        ws = guard.alloc(lbt.workspace_bytes(lbt.OP_GEMM_WGRAD, desc), torch.uint8)
        dW = guard.alloc((O, I), torch.float32, float("nan"))
        accW = guard.alloc((O, I), torch.int32, -77)
        lbt.qgemm_wgrad(q_dY, q_X, _sptr(sc, 0), _sptr(sc, 2), dW, accW, M, O, I, bits_g, 4, ws, status)
        _status_ok(status)
        _check_out(dW, accW, ref.gemm_backward("wgrad", c_dY, c_X, M, O, I, threads=threads), S_G, S_X)
    guard.check()


# Shapes whose output has more tiles than the persistent kernels have CTAs (148) or CTA pairs (74), so that
# every CTA walks several tiles: accumulator-buffer swaps, ring phases carried across tiles, banded tile order.
PERSISTENT = [
    (4096, 256, 2048, ("dgrad", "wgrad")),   # dgrad: 16 x 8 = 128 pair tiles; wgrad: 8 pair tiles x 9 reduction slices
    (512, 2048, 2560, ("wgrad",)),           # wgrad: 8 x 10 = 80 pair tiles, unsplit reduction
    (25600, 64, 96, ("dgrad", "wgrad")),     # dgrad: 200 single-CTA tiles of 128 x 96
    (128, 19200, 64, ("wgrad",)),            # wgrad: 150 single-CTA tiles
    (9500, 200, 384, ("dgrad",)),            # dgrad: 38 x 2 pair tiles, ragged in rows, columns and reduction
    (20224, 200, 256, ("dgrad",)),           # dgrad: 79 pair tiles = one round + 5: the 5 are cut into 4 column slices each
    (24064, 72, 256, ("dgrad",)),            # dgrad: 94 pair tiles = one round + 20: too many left over to cut
    (19300, 136, 272, ("dgrad",)),           # the same with ragged rows and a second, mostly empty column tile
]


@pytest.mark.parametrize("M,O,I,kinds", PERSISTENT, ids=lambda v: str(v))
def test_linear_layer_with_several_tiles_per_cta(M, O, I, kinds):
    dy = _codes_for(M * O, 4, True, 7, 0)
    w = _codes_for(O * I, 4, True, 7, 1)
    x = _codes_for(M * I, 4, False, 7, 2)
    _linear_backward_exhaustive(M, O, I, 4, dy, w, x, kinds, threads=THREADS)


def test_linear_without_accumulator_output_and_split_reduction():
    M, O, I = 4096, 64, 48          # a long reduction over few output tiles: wgrad splits it
    q_dY, c_dY = _codes_for(M * O, 4, True, 2, 0)
    q_X, c_X = _codes_for(M * I, 4, False, 2, 2)
    sc = _scales()
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_GEMM_WGRAD, lbt.GemmDesc(M, O, I)), dtype=torch.uint8, device="cuda")
    dW = torch.full((O, I), float("nan"), device="cuda")
    lbt.qgemm_wgrad(q_dY, q_X, _sptr(sc, 0), _sptr(sc, 2), dW, None, M, O, I, 4, 4, ws)
    torch.cuda.synchronize()
    want, _ = ref.epilogue(ref.gemm_backward("wgrad", c_dY, c_X, M, O, I), S_G, S_X)
    assert np.array_equal(dW.cpu().numpy(), want)


CONVS = [
    dict(N=2, C=3, H=5, W=5, K=4, R=3, S=3, stride=1, pad=1),
    dict(N=2, C=2, H=6, W=6, K=3, R=3, S=3, stride=2, pad=1),
    dict(N=1, C=3, H=9, W=9, K=2, R=7, S=7, stride=2, pad=3),
    dict(N=3, C=4, H=4, W=6, K=5, R=1, S=1, stride=1, pad=0),
    dict(N=2, C=4, H=6, W=6, K=3, R=1, S=1, stride=2, pad=0),
    dict(N=1, C=2, H=5, W=7, K=2, R=3, S=3, stride=1, pad=0),
    dict(N=1, C=1, H=6, W=5, K=1, R=2, S=3, stride=2, pad=1),
    dict(N=3, C=20, H=7, W=7, K=40, R=3, S=3, stride=1, pad=1),
    dict(N=4, C=16, H=14, W=14, K=32, R=3, S=3, stride=2, pad=1),
    dict(N=2, C=3, H=32, W=32, K=16, R=7, S=7, stride=2, pad=3),
    dict(N=2, C=144, H=6, W=6, K=272, R=3, S=3, stride=1, pad=1),
    dict(N=8, C=16, H=32, W=32, K=16, R=3, S=3, stride=1, pad=1),
]


def _run_conv(shape, bits_g=4, want_acc=True):
    d = ref.ConvShape(**shape)
    desc = lbt.ConvDesc(**shape)
    q_dY, c_dY = _codes_for(d.N * d.P * d.Q * d.K, bits_g, True, 3, 0)
    q_W, c_W = _codes_for(d.K * d.R * d.S * d.C, 4, True, 3, 1)
    q_X, c_X = _codes_for(d.N * d.H * d.W * d.C, 4, False, 3, 2)
    sc = _scales()
    guard = Guard()
    ws = guard.alloc(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), torch.uint8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dX = guard.alloc((d.N, d.H, d.W, d.C), torch.float32, float("nan"))
    dW = guard.alloc((d.K, d.R, d.S, d.C), torch.float32, float("nan"))
    accX = guard.alloc(dX.shape, torch.int32, -77) if want_acc else None
    accW = guard.alloc(dW.shape, torch.int32, -77) if want_acc else None
    lbt.qconv_dgrad_wgrad(desc, q_dY, q_W, q_X, _sptr(sc, 0), _sptr(sc, 1), _sptr(sc, 2), dX, dW, accX, accW,
                          bits_g, 4, 4, ws, status)
    _status_ok(status)
    guard.check()
    return d, (c_dY, c_W, c_X), (dX, dW, accX, accW)


@pytest.mark.parametrize("shape", CONVS, ids=lambda s: "N{N}C{C}H{H}K{K}R{R}s{stride}p{pad}".format(**s))
def test_convolution(shape):
    d, (c_dY, c_W, c_X), (dX, dW, accX, accW) = _run_conv(shape)
    _check_out(dX, accX, ref.conv_backward("dgrad", d, c_dY, c_W, threads=8), S_G, S_W)
    _check_out(dW, accW, ref.conv_backward("wgrad", d, c_dY, c_X, threads=8), S_G, S_X)


# Convolutions that keep the persistent kernels busy for three rounds or more, compared exhaustively.
PERSISTENT_CONVS = [
    # CTA-pair kernel, row window shared by the nine taps: 170 x 15 x 15 grid cells = 150 pair tiles on 74 pairs;
    # 160 gradient channels make the second reduction chunk of every tap ragged (32 of 128 bytes)
    dict(N=170, C=256, H=14, W=14, K=160, R=3, S=3, stride=1, pad=1),
    # single-CTA kernel, window + resident filter: 40 x 34 x 34 cells = 362 tiles on 148 SMs; multi-tap wgrad groups
    dict(N=40, C=64, H=32, W=32, K=64, R=3, S=3, stride=1, pad=1),
    # stride 2 on CTA pairs: four parity classes x 2 column tiles, one box per tap
    dict(N=96, C=320, H=14, W=14, K=144, R=3, S=3, stride=2, pad=1),
]


@pytest.mark.parametrize("shape", PERSISTENT_CONVS, ids=lambda s: "N{N}C{C}H{H}K{K}R{R}s{stride}p{pad}".format(**s))
def test_convolution_with_several_tiles_per_cta(shape):
    d, (c_dY, c_W, c_X), (dX, dW, accX, accW) = _run_conv(shape)
    _check_out(dX, accX, ref.conv_backward("dgrad", d, c_dY, c_W, threads=THREADS), S_G, S_W)
    _check_out(dW, accW, ref.conv_backward("wgrad", d, c_dY, c_X, threads=THREADS), S_G, S_X)


def test_convolution_eight_bit_gradients_without_accumulators():
    d, (c_dY, c_W, c_X), (dX, dW, _, _) = _run_conv(CONVS[8], bits_g=8, want_acc=False)
    want, _ = ref.epilogue(ref.conv_backward("dgrad", d, c_dY, c_W), S_G, S_W)
    assert np.array_equal(dX.cpu().numpy(), want)
    want, _ = ref.epilogue(ref.conv_backward("wgrad", d, c_dY, c_X), S_G, S_X)
    assert np.array_equal(dW.cpu().numpy(), want)


def test_host_side_rejections():
    L = lbt.lib()
    sc = _scales()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    out = torch.zeros(1 << 12, device="cuda")
    p, o = buf.data_ptr(), out.data_ptr()
    call = lambda M, O, I, bg, bw, ws, wsb: L.lbt_qgemm_dgrad(p, p, _sptr(sc, 0), _sptr(sc, 1), o, None, M, O, I, bg, bw,
                                                          None, ws, wsb, 0)
    need = lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, lbt.GemmDesc(8, 8, 8))
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    assert call(8, 8, 8, 4, 4, ws.data_ptr(), need - 1) == lbt.ERR_WORKSPACE
    assert call(8, 8, 8, 4, 4, None, 0) == lbt.ERR_WORKSPACE
    assert call(8, 8, 8, 9, 4, ws.data_ptr(), need) == lbt.ERR_UNSUPPORTED_BITS
    assert call(0, 8, 8, 4, 4, ws.data_ptr(), need) == lbt.ERR_INVALID_ARG
    assert call(8, 1 << 20, 8, 8, 8, ws.data_ptr(), need) in (lbt.ERR_ACC_RANGE, lbt.ERR_WORKSPACE)
    big = lbt.ConvDesc(N=256, C=3, H=224, W=224, K=64, R=7, S=7, stride=2, pad=3)
    assert L.lbt_qconv_dgrad_wgrad(ctypes.addressof(big), p, p, p, _sptr(sc, 0), _sptr(sc, 1), _sptr(sc, 2), None, o,
                                   None, None, 8, 4, 4, None, ws.data_ptr(), 1 << 40, 0) == lbt.ERR_ACC_RANGE
    bad = lbt.ConvDesc(N=1, C=1, H=8, W=8, K=1, R=3, S=3, stride=3, pad=1)
    assert lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, bad) == 0


def test_outputs_aligned_to_16_but_not_to_32_bytes():
    """The epilogue stores whole 32-byte sectors where the output rows allow it; buffers that are only 16-byte
    aligned (the documented minimum) must take the other path and give the same results."""
    shape = dict(N=3, C=24, H=7, W=7, K=40, R=3, S=3, stride=1, pad=1)
    d, desc = ref.ConvShape(**shape), lbt.ConvDesc(**shape)
    q_dY, c_dY = _codes_for(d.N * d.P * d.Q * d.K, 4, True, 9, 0)
    q_W, c_W = _codes_for(d.K * d.R * d.S * d.C, 4, True, 9, 1)
    q_X, c_X = _codes_for(d.N * d.H * d.W * d.C, 4, False, 9, 2)
    sc = _scales()
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    nx, nw = d.N * d.H * d.W * d.C, d.K * d.R * d.S * d.C

    def shifted(n, dtype, fill):          # starts 16 bytes into an allocation
        buf = torch.full((n + 8,), fill, dtype=dtype, device="cuda")
        view = buf[4:4 + n]
        assert view.data_ptr() % 32 == 16
        return buf, view

    bx, dX = shifted(nx, torch.float32, float("nan"))
    bw, dW = shifted(nw, torch.float32, float("nan"))
    bax, accX = shifted(nx, torch.int32, -77)
    baw, accW = shifted(nw, torch.int32, -77)
    lbt.qconv_dgrad_wgrad(desc, q_dY, q_W, q_X, _sptr(sc, 0), _sptr(sc, 1), _sptr(sc, 2), dX, dW, accX, accW, 4, 4, 4, ws, status)
    _status_ok(status)
    _check_out(dX, accX, ref.conv_backward("dgrad", d, c_dY, c_W), S_G, S_W)
    _check_out(dW, accW, ref.conv_backward("wgrad", d, c_dY, c_X), S_G, S_X)
    for buf in (bax, baw):                # the four elements before and after stay untouched
        assert (buf[:4] == -77).all() and (buf[-4:] == -77).all()
    for buf in (bx, bw):
        assert torch.isnan(buf[:4]).all() and torch.isnan(buf[-4:]).all()
