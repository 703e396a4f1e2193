"""The batch-sharded backward pass through a live communicator: two processes share cuda:0, each holds
one slice of the batch on the device and calls `dp.sharded_backward(..., comm=DistComm())`; the
collectives are real `torch.distributed` all-reduces on the device tensors (gloo backend: it stages
CUDA tensors through the host, so two ranks can share one GPU; the ranks meet on the host only, no
kernel of one rank waits for a kernel of the other).  Every rank's codes, statistics, gamma, dX and
the int32 / fp32 weight gradient must equal the oracle on the WHOLE batch bit for bit -- also when the
caller passes a stream that is not torch's current one."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import ref
from paper_2407_12637_b200 import lbt, synth

pytestmark = pytest.mark.gpu

S_W, S_X = 0.01, 0.05
GAMMA, SEED, ITER = 0.7, 3, 5


def _whole_batch(shape, bits_g):
    """Seeded inputs of the whole layer (host arrays): the parent and every rank draw the same."""
    d = ref.ConvShape(**shape)
    dY = synth.laplace_outliers(d.N * d.P * d.Q * d.K, 1e-3, SEED)
    raw_w = synth.code_bytes((d.K * d.R * d.S * d.C + 1) // 2, SEED, 1)
    raw_x = synth.code_bytes(d.N * d.H * d.W * d.C // 2, SEED, 2)
    return d, dY, raw_w, raw_x


def _rank_main(rank, world, port, shape, splits, bits_g, side_stream, out):
    import torch.distributed as dist
    from paper_2407_12637_b200 import dp
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        d, dY_all, raw_w, raw_x_all = _whole_batch(shape, bits_g)
        per_y, per_x = d.P * d.Q * d.K, d.H * d.W * d.C
        img0, m = sum(splits[:rank]), splits[rank]
        offsets = dp.shard_offsets([k * per_y for k in splits])
        assert (img0 * per_x) % 2 == 0
        desc = lbt.ConvDesc(**{**shape, "N": m})
        dY = torch.from_numpy(dY_all[img0 * per_y:(img0 + m) * per_y]).cuda()
        q_W = torch.from_numpy(raw_w).cuda()
        q_X = torch.from_numpy(raw_x_all[img0 * per_x // 2:(img0 + m) * per_x // 2]).cuda()
        sc = torch.tensor([S_W, S_X], dtype=torch.float32, device="cuda")
        state = lbt.new_state(gamma=GAMMA, bits=bits_g, rounding=lbt.ROUND_STOCHASTIC, seed=SEED, it=ITER)
        stats = lbt.new_stats()
        q_dY = torch.empty((dY.numel() + 1) // 2 if bits_g <= 4 else dY.numel(), dtype=torch.uint8, device="cuda")
        dX = torch.full((m, d.H, d.W, d.C), float("nan"), device="cuda")
        dW = torch.full((d.K, d.R, d.S, d.C), float("nan"), device="cuda")
        accW = torch.full(dW.shape, -77, dtype=torch.int32, device="cuda")
        ws = torch.empty(lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, desc), dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        stream = torch.cuda.Stream() if side_stream else None     # NOT made current by the caller
        dp.sharded_backward(desc, dY, q_W, q_X, sc.data_ptr(), sc.data_ptr() + 4, state, stats, q_dY, dX, dW, accW,
                            bits_g, ws, index_offset=offsets[rank], images_total=d.N, comm=dp.DistComm(), stream=stream)
        (stream or torch.cuda.current_stream()).synchronize()
        out.put((rank, {k: v.cpu().numpy() for k, v in
                        dict(state=state, stats=stats, q_dY=q_dY, dX=dX, dW=dW, accW=accW).items()}))
        dist.barrier()
    finally:
        dist.destroy_process_group()


CASES = [
    (dict(N=6, C=16, H=8, W=8, K=24, R=3, S=3, stride=1, pad=1), [2, 4], 4, False),
    (dict(N=6, C=16, H=8, W=8, K=24, R=3, S=3, stride=1, pad=1), [4, 2], 4, True),
    (dict(N=384, C=144, H=1, W=1, K=272, R=1, S=1, stride=1, pad=0), [128, 256], 8, True),
]


@pytest.mark.parametrize("shape,splits,bits_g,side_stream", CASES,
                         ids=["conv3x3_current_stream", "conv3x3_side_stream", "linear_8bit_side_stream"])
def test_two_ranks_on_device_tensors_match_the_whole_batch_oracle(shape, splits, bits_g, side_stream):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    world = len(splits)
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, shape, splits, bits_g, side_stream, out))
             for r in range(world)]
    for p in procs:
        p.start()
    try:
        results = dict(out.get(timeout=300) for _ in procs)
    finally:
        for p in procs:
            p.join(timeout=120)
            if p.is_alive():
                p.kill()
    assert all(p.exitcode == 0 for p in procs)

    d, dY, raw_w, raw_x = _whole_batch(shape, bits_g)
    c_W = ref.unpack4(raw_w, d.K * d.R * d.S * d.C, True)
    c_X = ref.unpack4(raw_x, d.N * d.H * d.W * d.C, False)
    g_max, bad = ref.grad_stats(dY)
    q = ref.quantize_grad(dY, GAMMA, g_max, bits_g, rounding=1, seed=SEED, it=ITER)
    gamma = ref.update_interval(GAMMA, 1e-3, 1e-3, 1e-3, 1.0, bits_g, dY.size, q.n_out, bad)
    accX = ref.conv_backward("dgrad", d, q.codes, c_W, threads=8)
    accW = ref.conv_backward("wgrad", d, q.codes, c_X, threads=8)
    wantX, _ = ref.epilogue(accX, q.scale, S_W)
    wantW, _ = ref.epilogue(accW, q.scale, S_X)
    per_y = d.P * d.Q * d.K
    for rank, r in results.items():
        st = lbt.IntervalState.from_buffer_copy(r["state"].tobytes())
        gs = lbt.GradStats.from_buffer_copy(r["stats"].tobytes())
        img0, m = sum(splits[:rank]), splits[rank]
        assert st.dev_status == 0 and st.iter == ITER + 1 and np.float32(st.gamma) == np.float32(gamma)
        assert (gs.g_max, gs.n, gs.n_out, gs.n_nonfinite) == (g_max, dY.size, q.n_out, 0)
        assert np.float32(gs.scale) == q.scale
        assert np.array_equal(r["q_dY"], ref.pack(q.codes[img0 * per_y:(img0 + m) * per_y], bits_g))
        assert np.array_equal(r["dX"], wantX[img0:img0 + m])
        assert np.array_equal(r["accW"], accW.astype(np.int32))
        assert np.array_equal(r["dW"], wantW)
