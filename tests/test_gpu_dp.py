"""GPU parity of the batch-sharded backward pass: R ranks' phases run one after another on one GPU,
with the reductions between them done in place of the collectives; codes, statistics, gamma, dX and
the int32 / fp32 weight gradient must equal the oracle's (and hence the one-GPU call's) bit for bit."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import dp, lbt, synth
from tests.test_gpu_contractions import _codes_for

pytestmark = pytest.mark.gpu

S_W, S_X = 0.01, 0.05


class _Shard:
    pass


def _run_sharded(shape, splits, bits_g, rounding, seed):
    """splits: images per rank.  Returns the per-rank buffers after all four phases."""
    d_all = ref.ConvShape(**shape)
    n_img = d_all.N
    assert sum(splits) == n_img
    per_img_y = d_all.P * d_all.Q * d_all.K
    per_img_x = d_all.H * d_all.W * d_all.C
    dY_all = synth.laplace_outliers(n_img * per_img_y, 1e-3, seed)
    q_W, c_W = _codes_for(d_all.K * d_all.R * d_all.S * d_all.C, 4, True, seed, 1)
    _, c_X = _codes_for(n_img * per_img_x, 4, False, seed, 2)
    sc = torch.tensor([S_W, S_X], dtype=torch.float32, device="cuda")
    offs = dp.shard_offsets([m * per_img_y for m in splits])
    shards, img0 = [], 0
    for r, m in enumerate(splits):
        s = _Shard()
        s.desc = lbt.ConvDesc(**{**shape, "N": m})
        s.dY = torch.from_numpy(dY_all[img0 * per_img_y:(img0 + m) * per_img_y]).cuda()
        x_codes = c_X[img0 * per_img_x:(img0 + m) * per_img_x]
        assert (img0 * per_img_x) % 2 == 0
        s.q_X = torch.from_numpy(_pack_unsigned(x_codes)).cuda()
        s.state = lbt.new_state(gamma=0.7, alpha=1e-3, beta=1e-3, bits=bits_g, rounding=rounding, seed=seed, it=5)
        s.stats = lbt.new_stats()
        s.q_dY = torch.empty((s.dY.numel() + 1) // 2 if bits_g <= 4 else s.dY.numel(), dtype=torch.uint8, device="cuda")
        s.dX = torch.full((m, d_all.H, d_all.W, d_all.C), float("nan"), device="cuda")
        s.dW = torch.full((d_all.K, d_all.R, d_all.S, d_all.C), float("nan"), device="cuda")
        s.accW = torch.full(s.dW.shape, -77, dtype=torch.int32, device="cuda")
        s.ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, s.desc), dtype=torch.uint8, device="cuda")
        s.offset, s.img0 = offs[r], img0
        shards.append(s)
        img0 += m
    dp.check_acc_range(shards[0].desc, n_img, bits_g, 4)
    # phase 1 + "all-reduce": max of g_max, sums of the counters
    for s in shards:
        dp.phase_stats(s.dY, s.state, s.stats)
    g = torch.stack([s.stats[0:4].view(torch.float32) for s in shards]).max(dim=0).values
    cnt = torch.stack([s.stats[16:40].view(torch.int64) for s in shards]).sum(dim=0)
    for s in shards:
        s.stats[0:4].view(torch.float32).copy_(g)
        s.stats[16:40].view(torch.int64).copy_(cnt)
    # phase 2 + sum of n_out
    for s in shards:
        dp.phase_quantize(s.dY, s.offset, s.state, s.stats, s.q_dY)
    n_out = torch.stack([s.stats[24:32].view(torch.int64) for s in shards]).sum(dim=0)
    for s in shards:
        s.stats[24:32].view(torch.int64).copy_(n_out)
    # phase 3 + sum of the integer accumulators, phase 4
    for s in shards:
        dp.phase_contract(s.desc, s.q_dY, q_W, s.q_X, sc.data_ptr(), sc.data_ptr() + 4, s.state, s.stats,
                          s.dX, s.dW, s.accW, bits_g, s.ws)
    acc = torch.stack([s.accW for s in shards]).sum(dim=0, dtype=torch.int32)
    for s in shards:
        s.accW.copy_(acc)
        dp.phase_finalize(s.accW, s.stats, sc.data_ptr() + 4, s.dW)
    torch.cuda.synchronize()
    return d_all, dY_all, c_W, c_X, shards


def _pack_unsigned(codes):
    c = codes.astype(np.uint8)
    if c.size % 2:
        c = np.concatenate([c, np.zeros(1, np.uint8)])
    return (c[0::2] | (c[1::2] << 4)).astype(np.uint8)


CASES = [
    (dict(N=6, C=16, H=8, W=8, K=24, R=3, S=3, stride=1, pad=1), [2, 4], 4, lbt.ROUND_STOCHASTIC),
    (dict(N=6, C=16, H=8, W=8, K=24, R=3, S=3, stride=1, pad=1), [1, 2, 3], 4, lbt.ROUND_NEAREST),
    (dict(N=8, C=20, H=9, W=9, K=40, R=3, S=3, stride=2, pad=1), [3, 5], 8, lbt.ROUND_STOCHASTIC),
    (dict(N=384, C=144, H=1, W=1, K=272, R=1, S=1, stride=1, pad=0), [128, 256], 4, lbt.ROUND_STOCHASTIC),
]


@pytest.mark.parametrize("shape,splits,bits_g,rounding", CASES,
                         ids=["conv3x3_2ranks_sr4", "conv3x3_3ranks_nearest4", "conv3x3s2_2ranks_sr8", "linear_2ranks_sr4"])
def test_sharded_backward_equals_the_unsharded_oracle(shape, splits, bits_g, rounding):
    d, dY, c_W, c_X, shards = _run_sharded(shape, splits, bits_g, rounding, seed=3)
    # the oracle on the WHOLE batch
    g_max, bad = ref.grad_stats(dY)
    q = ref.quantize_grad(dY, 0.7, g_max, bits_g, rounding=rounding, seed=3, it=5)
    gamma = ref.update_interval(0.7, 1e-3, 1e-3, 1e-3, 1.0, bits_g, dY.size, q.n_out, bad)
    accX = ref.conv_backward("dgrad", d, q.codes, c_W, threads=8)
    accW = ref.conv_backward("wgrad", d, q.codes, c_X, threads=8)
    wantX, _ = ref.epilogue(accX, q.scale, S_W)
    wantW, _ = ref.epilogue(accW, q.scale, S_X)
    per_img_y = d.P * d.Q * d.K
    for s in shards:
        st, gs = lbt.read_state(s.state), lbt.read_stats(s.stats)
        assert st.dev_status == 0 and st.iter == 6
        assert (gs.g_max, gs.n, gs.n_out, gs.n_nonfinite) == (g_max, dY.size, q.n_out, 0)
        assert np.float32(gs.scale) == q.scale and np.float32(st.gamma) == np.float32(gamma)
        m = s.desc.N
        want_codes = q.codes[s.img0 * per_img_y:(s.img0 + m) * per_img_y]
        assert np.array_equal(s.q_dY.cpu().numpy(), ref.pack(want_codes, bits_g))
        assert np.array_equal(s.dX.cpu().numpy(), wantX[s.img0:s.img0 + m])
        assert np.array_equal(s.accW.cpu().numpy(), accW.astype(np.int32))
        assert np.array_equal(s.dW.cpu().numpy(), wantW)


def test_single_rank_sharded_call_equals_the_fused_call():
    """`sharded_backward` without a communicator is the fused `qconv_backward`."""
    shape = dict(N=4, C=16, H=8, W=8, K=32, R=3, S=3, stride=1, pad=1)
    d = ref.ConvShape(**shape)
    desc = lbt.ConvDesc(**shape)
    dY = torch.from_numpy(synth.laplace_outliers(d.N * d.P * d.Q * d.K, 1e-3, 9)).cuda()
    q_W, _ = _codes_for(d.K * d.R * d.S * d.C, 4, True, 9, 1)
    q_X, _ = _codes_for(d.N * d.H * d.W * d.C, 4, False, 9, 2)
    sc = torch.tensor([S_W, S_X], dtype=torch.float32, device="cuda")
    outs = []
    for sharded in (False, True):
        st = lbt.new_state(gamma=0.6, bits=4, rounding=lbt.ROUND_STOCHASTIC, seed=2, it=1)
        stats = lbt.new_stats()
        q_dY = torch.empty(dY.numel() // 2, dtype=torch.uint8, device="cuda")
        dX = torch.empty(d.N, d.H, d.W, d.C, device="cuda")
        dW = torch.empty(d.K, d.R, d.S, d.C, device="cuda")
        accW = torch.empty(dW.shape, dtype=torch.int32, device="cuda")
        ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")
        if sharded:
            dp.sharded_backward(desc, dY, q_W, q_X, sc.data_ptr(), sc.data_ptr() + 4, st, stats, q_dY, dX, dW, accW,
                                4, ws, index_offset=0, images_total=d.N, comm=None)
        else:
            lbt.qconv_backward(desc, dY, q_W, q_X, sc.data_ptr(), sc.data_ptr() + 4, st, stats, q_dY, dX, dW, None,
                               accW, 4, ws)
        torch.cuda.synchronize()
        outs.append([t.cpu().numpy().copy() for t in (st, stats, q_dY, dX, dW, accW)])
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_shard_offset_must_be_a_multiple_of_eight():
    L = lbt.lib()
    buf = torch.zeros(256, device="cuda")
    st, stats = lbt.new_state(), lbt.new_stats()
    p = buf.data_ptr()
    assert L.lbt_quantize_grad_shard(p, 64, 12, st.data_ptr(), stats.data_ptr(), p, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_dequantize_acc(p, 8, None, p, p, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_dequantize_acc(p + 4, 8, p, p, p, 0) == lbt.ERR_ALIGNMENT
