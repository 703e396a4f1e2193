"""Two gloo ranks on CPU: the benchmark's multi-process aggregation (max time over ranks, summed units)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2407_12637_b200 import dist_util


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 2.0 if rank == 0 else 5.0                      # rank 1 is the slow one
    out.put((rank, dist_util.max_over_ranks(ms), dist_util.aggregate_throughput(10.0, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_work():
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
    for _rank, worst, tput in results:
        assert worst == 5.0
        assert tput == 2 * 10.0 / 5e-3


def test_single_process_is_the_identity():
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.aggregate_throughput(7.0, 2.0) == 7.0 / 2e-3
