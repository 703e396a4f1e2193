"""Host logic of the batch-sharded backward pass on CPU: shard offsets, the accumulator-range check,
and (two gloo ranks) the reductions of the statistics struct and of integer accumulators."""
import ctypes
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2407_12637_b200 import dp, lbt


def _stats_bytes(g_max, n, n_out, n_nonfinite):
    s = lbt.GradStats(g_max, 0.0, 0.0, 0, n, n_out, n_nonfinite)
    return torch.frombuffer(bytearray(bytes(s)), dtype=torch.uint8).clone()


def _read(t):
    return lbt.GradStats.from_buffer_copy(t.numpy().tobytes())


def test_shard_offsets_are_prefix_sums_and_block_aligned():
    assert dp.shard_offsets([16, 8, 24]) == [0, 16, 24]
    assert dp.shard_offsets([40]) == [0]
    with pytest.raises(ValueError):
        dp.shard_offsets([12, 8])          # the second shard would start inside a block of eight


def test_accumulator_range_is_checked_for_the_whole_batch():
    d = lbt.ConvDesc(N=64, C=64, H=56, W=56, K=64, R=3, S=3, stride=1, pad=1)
    dp.check_acc_range(d, 256, 4, 4)                      # 256 * 3136 * 8 * 15 < 2^31
    with pytest.raises(lbt.LbtError):
        dp.check_acc_range(d, 256, 8, 8)                  # 256 * 3136 * 128 * 255 does not fit


def test_struct_field_offsets_match_the_slices():
    assert lbt.GradStats.g_max.offset == 0 and lbt.GradStats.n.offset == 16
    assert lbt.GradStats.n_out.offset == 24 and lbt.GradStats.n_nonfinite.offset == 32
    assert ctypes.sizeof(lbt.GradStats) == 40


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    comm = dp.DistComm()
    stats = _stats_bytes([0.25, 3.5][rank], [1000, 24][rank], 0, [0, 2][rank])
    dp.reduce_stats(stats, comm)
    after_absmax = _read(stats)
    local_out = [7, 11][rank]
    stats[24:32] = torch.from_numpy(np.array([local_out], np.int64).view(np.uint8))
    dp.reduce_n_out(stats, comm)
    after_quant = _read(stats)
    acc = torch.tensor([[2 ** 29, -5, rank], [7, -(2 ** 29), 1]], dtype=torch.int32)
    comm.all_reduce(acc, "sum")
    out.put((rank, (after_absmax.g_max, after_absmax.n, after_absmax.n_out, after_absmax.n_nonfinite),
             (after_quant.g_max, after_quant.n, after_quant.n_out, after_quant.n_nonfinite), acc.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_statistics_and_integer_accumulators():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _rank, a, b, acc in results:
        assert a == (3.5, 1024, 0, 2)                     # max of g_max; sums of n, n_nonfinite; n_out still 0
        assert b == (3.5, 1024, 18, 2)                    # only n_out changes in the second reduction
        assert acc == [[2 ** 30, -10, 1], [14, -(2 ** 30), 2]]   # integer sums: exact, order-free


def test_single_rank_needs_no_communicator():
    stats = _stats_bytes(1.5, 80, 3, 0)
    before = stats.clone()
    dp.reduce_stats(stats, None)
    dp.reduce_n_out(stats, None)
    assert torch.equal(stats, before)
