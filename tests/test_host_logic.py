"""Host-side logic of the C-ABI library that needs no GPU: argument validation happens before any
CUDA call, and the workspace size follows the padded cell grid described in the design notes."""
import ctypes

import pytest

from paper_2407_12637_b200 import build as lib_build
from paper_2407_12637_b200 import lbt, shapes


@pytest.fixture(scope="module")
def L():
    lib_build.build()
    return lbt.lib()


def _up(v, a):
    return (v + a - 1) // a * a


def _grid(d):
    """Python restatement of the cell-grid geometry: per image Hg x Wg cells."""
    st, pad = d["stride"], d["pad"]
    P = (d["H"] + 2 * pad - d["R"]) // st + 1
    Q = (d["W"] + 2 * pad - d["S"]) // st + 1

    def halo(taps):
        offs = [(r - pad) // st for r in range(taps)]                       # wgrad (floor division)
        offs += [(ph + pad - r) // st for r in range(taps) for ph in range(st) if (ph + pad - r) % st == 0]
        return max(max(offs), -min(offs), 0)

    Hg = max(P, -(-d["H"] // st)) + halo(d["R"])
    Wg = max(Q, -(-d["W"] // st)) + halo(d["S"])
    return P, Q, Hg, Wg


def _wgrad_tile_columns(d, Kp, Cp, Wg):
    """Tiles per filter: one per tap, or (narrow layers, multi-tap tiles) one per group of taps that read
    the same parity class of X at row offsets at most 128 apart, at most 512 / round_up(Cp, 32) (<= 16) taps."""
    st, pad = d["stride"], d["pad"]
    taps = [(((r - pad) % st) * st + (s - pad) % st, ((r - pad) // st) * Wg + (s - pad) // st)
            for r in range(d["R"]) for s in range(d["S"])]
    if Cp > 128 or Kp > 128 or len(taps) < 2:
        return len(taps)
    taps.sort()
    most = min(512 // _up(Cp, 32), 16)
    groups, i, run_end, cap, largest = 0, 0, 0, most, 0
    while i < len(taps):
        if i >= run_end:                                   # a new class: its taps spread evenly over the fewest groups
            run_end = i + 1
            while run_end < len(taps) and taps[run_end][0] == taps[i][0]:
                run_end += 1
            n = run_end - i
            cap = -(-n // -(-n // most))
        j = i + 1
        while j < run_end and j - i < cap and taps[j][1] - taps[i][1] <= 128:
            j += 1
        groups += 1
        largest = max(largest, j - i)
        i = j
    return groups if 10 * len(taps) >= 7 * largest * groups else len(taps)   # too unbalanced: one tile per tap


@pytest.mark.parametrize("d", [shapes.conv(256, 256, 14, 14, 256, 3, 3, 1, 1), shapes.conv(256, 3, 224, 224, 64, 7, 7, 2, 3),
                               shapes.conv(256, 64, 56, 56, 128, 1, 1, 2, 0), shapes.conv(2, 5, 9, 7, 3, 3, 3, 2, 1),
                               shapes.linear(8192, 8192, 8192), shapes.linear(5, 3, 7)],
                         ids=lambda d: "N{N}C{C}H{H}K{K}R{R}s{stride}".format(**d))
def test_workspace_follows_the_cell_grid(L, d):
    fwd, bwd = _workspace(d)
    if d["C"] < 8 and d["R"] * d["S"] > 1:
        # very few input channels: forward and wgrad run as the linear layer over explicit patches
        lin = shapes.linear(d["N"] * _grid(d)[0] * _grid(d)[1], d["K"], d["R"] * d["S"] * d["C"])
        fwd, bwd = max(fwd, _workspace(lin)[0]), max(bwd, _workspace(lin)[1])
    assert lbt.workspace_bytes(lbt.OP_CONV_FORWARD, lbt.ConvDesc(**d)) == fwd
    assert lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, lbt.ConvDesc(**d)) == bwd


def _workspace(d):
    P, Q, Hg, Wg = _grid(d)
    rows = d["N"] * Hg * Wg
    Kp, Cp, st2 = _up(d["K"], 16), _up(d["C"], 16), d["stride"] ** 2
    want = 256 + _up(rows * Kp, 256) + _up(d["R"] * d["S"] * d["K"] * Cp, 256) + _up(st2 * rows * Cp, 256) + 256
    # wgrad adds one slab of int32 partial sums per slice of its split reduction (sized for 148 SMs)
    bn = 128 if Cp <= 128 else 256
    pair = bn == 256 and Kp > 128
    tiles = -(-Kp // (256 if pair else 128)) * _wgrad_tile_columns(d, Kp, Cp, Wg) * -(-Cp // bn)
    kb_total = -(-rows // 128)
    splits = max(1, min(kb_total, (74 if pair else 148) // tiles))
    splits = -(-kb_total // -(-kb_total // splits))
    part = _up(splits * _up(d["K"] * d["R"] * d["S"] * d["C"], 4) * 4, 256) if splits > 1 else 0
    return want, want + part


def test_known_grids():
    assert _grid(shapes.conv(1, 1, 14, 14, 1, 3, 3, 1, 1))[2:] == (15, 15)     # one shared halo row / column
    assert _grid(shapes.conv(1, 1, 224, 224, 1, 7, 7, 2, 3))[2:] == (114, 114)  # 112 + reach 2 of a 7-tap stride-2 filter
    assert _grid(shapes.conv(1, 1, 14, 14, 1, 1, 1, 1, 0))[2:] == (14, 14)      # pointwise: no padding at all
    assert _grid(shapes.linear(7, 3, 5))[2:] == (1, 1)


def test_invalid_descriptions_need_no_workspace(L):
    bad = [dict(N=0, C=1, H=1, W=1, K=1, R=1, S=1, stride=1, pad=0), dict(N=1, C=1, H=8, W=8, K=1, R=3, S=3, stride=3, pad=1),
           dict(N=1, C=1, H=2, W=2, K=1, R=5, S=5, stride=1, pad=0), dict(N=1, C=1, H=8, W=8, K=1, R=9, S=9, stride=1, pad=4),
           dict(N=1, C=1, H=8, W=8, K=1, R=3, S=3, stride=1, pad=-1)]
    for d in bad:
        assert lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, lbt.ConvDesc(**d)) == 0
    assert lbt.workspace_bytes(lbt.OP_GEMM_WGRAD, lbt.GemmDesc(1, 1, 0)) == 0
    assert lbt.workspace_bytes(99, lbt.GemmDesc(1, 1, 1)) == 0
    assert lbt.workspace_bytes(lbt.OP_QUANTIZE) == 0


def test_rejections_before_any_cuda_call(L):
    """Every check below fails on the host, so none of these calls reaches the GPU (pointers are fakes)."""
    p = 0x10000          # any 16-byte aligned non-null value
    big = 1 << 40
    assert L.lbt_qgemm_dgrad(p, p, p, p, p, None, 0, 8, 8, 4, 4, None, p, big, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_qgemm_dgrad(p, p, p, p, None, None, 8, 8, 8, 4, 4, None, p, big, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_qgemm_dgrad(p, None, p, p, p, None, 8, 8, 8, 4, 4, None, p, big, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_qgemm_dgrad(p, p, p, p, p, None, 8, 8, 8, 1, 4, None, p, big, 0) == lbt.ERR_UNSUPPORTED_BITS
    assert L.lbt_qgemm_wgrad(p, p, p, p, p, None, 8, 8, 8, 4, 9, None, p, big, 0) == lbt.ERR_UNSUPPORTED_BITS
    assert L.lbt_qgemm_dgrad(p + 4, p, p, p, p, None, 8, 8, 8, 4, 4, None, p, big, 0) == lbt.ERR_ALIGNMENT
    assert L.lbt_qgemm_dgrad(p, p, p, p, p + 8, None, 8, 8, 8, 4, 4, None, p, big, 0) == lbt.ERR_ALIGNMENT
    assert L.lbt_qgemm_dgrad(p, p, p, p, p, None, 8, 8, 8, 4, 4, None, None, 0, 0) == lbt.ERR_WORKSPACE
    assert L.lbt_qgemm_dgrad(p, p, p, p, p, None, 8, 8, 8, 4, 4, None, p, 100, 0) == lbt.ERR_WORKSPACE
    # accumulator range: reduction length x largest |code| x largest |code| must stay below 2^31
    assert L.lbt_qgemm_dgrad(p, p, p, p, p, None, 8, 1 << 18, 8, 8, 8, None, p, big, 0) == lbt.ERR_ACC_RANGE   # 2^18 * 128 * 128
    assert L.lbt_qgemm_wgrad(p, p, p, p, p, None, 1 << 25, 8, 8, 4, 4, None, p, big, 0) == lbt.ERR_ACC_RANGE   # 2^25 * 8 * 15
    conv1 = lbt.ConvDesc(**shapes.CONFIG3["conv1"][0])
    call = lambda bits_g: L.lbt_qconv_dgrad_wgrad(ctypes.addressof(conv1), p, p, p, p, p, p, None, p, None, None,
                                                  bits_g, 4, 4, None, p, 0, 0)
    assert call(8) == lbt.ERR_ACC_RANGE           # 3.2 M x 128 x 15 > 2^31
    assert call(4) == lbt.ERR_WORKSPACE           # 3.2 M x 8 x 15 fits; the (zero-sized) workspace is what fails
    assert L.lbt_qconv_dgrad_wgrad(ctypes.addressof(conv1), p, p, p, p, p, p, None, None, None, None, 4, 4, 4, None,
                                   p, big, 0) == lbt.ERR_INVALID_ARG          # nothing to compute
    strided = lbt.ConvDesc(N=1, C=16, H=9, W=9, K=16, R=3, S=3, stride=3, pad=1)
    assert L.lbt_qconv_dgrad_wgrad(ctypes.addressof(strided), p, p, p, p, p, p, p, None, None, None, 4, 4, 4, None,
                                   p, big, 0) == lbt.ERR_UNSUPPORTED
    assert L.lbt_qconv_backward(ctypes.addressof(conv1), p, p, p, p, p, p, p, p, p, p, None, None, 11, p, big, 0) \
        == lbt.ERR_UNSUPPORTED_BITS
    assert L.lbt_qconv_backward(ctypes.addressof(conv1), None, p, p, p, p, p, p, p, p, p, None, None, 4, p, big, 0) \
        == lbt.ERR_INVALID_ARG
    assert L.lbt_qgemm_dgrad_static(p, p, p, p, p, None, 4096, 4096, 4096, 4, 4, None, 0) == lbt.ERR_SCRATCH_LIMIT
    assert L.lbt_set_timing_events(17, None, None) == lbt.ERR_INVALID_ARG
    assert L.lbt_set_timing_events(0, p, None) == lbt.ERR_INVALID_ARG
    assert L.lbt_selftest_wait_timeout(None, 5, 0) == lbt.ERR_INVALID_ARG
    for code in range(-10, 1):
        assert lbt.status_string(code).startswith("LBT_")
