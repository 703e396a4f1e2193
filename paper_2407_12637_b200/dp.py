"""Batch-sharded (data-parallel) backward pass of one layer that equals the one-GPU result bit for bit.

Every rank holds a slice of the batch (its rows of dY and X) and all of W.  The paper's per-layer
quantities span the whole batch (Sec. 3.1: g_max over all gradients of the layer; Sec. 3.3, Eq. 9:
the clip-out ratio), so they are reduced over the ranks, and the weight gradient is summed as
integers before the dequantising multiply, which makes the sum exact and order-free:

    phase_stats      local abs-max and counts            -> max of g_max, sum of n and n_nonfinite
    phase_quantize   codes with the whole tensor's random bits -> sum of n_out
    phase_contract   gamma update (same on every rank), dX of the slice, local int32 wgrad accumulators
                                                         -> sum of the accumulators
    phase_finalize   dW = (float)acc * fl32(s_g * s_x)

The collectives are plain `torch.distributed` all-reduces on fields of the device structs (NCCL on
GPUs); every arithmetic step runs in the library's kernels.  `comm` is any object with
`all_reduce(tensor, op)`; `DistComm` wraps a process group, `None` means a single rank.

Stream order: `torch.distributed` orders a collective against torch's CURRENT stream, the library
enqueues on the stream it is given.  `sharded_backward` therefore makes `stream` the current stream
for its whole body, so kernels and collectives form one sequence whatever stream the caller passes.
"""
from __future__ import annotations

import contextlib

import torch

from . import lbt

_G_MAX = slice(0, 4)        # float g_max
_DEV_STATUS = slice(lbt.IntervalState.dev_status.offset, lbt.IntervalState.dev_status.offset + 4)
_COUNTS = slice(16, 40)     # uint64 n, n_out, n_nonfinite (non-negative, far below 2^63: summed as int64)


class DistComm:
    """All-reduce over a `torch.distributed` process group (default group if None)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self._group = dist, group

    def all_reduce(self, tensor, op):
        red = self._dist.ReduceOp.MAX if op == "max" else self._dist.ReduceOp.SUM
        self._dist.all_reduce(tensor, op=red, group=self._group)


def shard_offsets(shard_elems):
    """Element index of each shard's first gradient in the whole tensor (batch-major order).  Every
    offset must be a multiple of 8: a stochastic-rounding block serves eight consecutive elements."""
    offs, total = [], 0
    for n in shard_elems:
        if total % 8:
            raise ValueError("a shard boundary splits a block of eight gradients: "
                             f"offset {total} is not a multiple of 8")
        offs.append(total)
        total += int(n)
    return offs


def reduce_stats(stats: torch.Tensor, comm) -> None:
    """After phase_stats: g_max <- max over ranks; n, n_nonfinite (and the still-zero n_out) <- sums."""
    if comm is None:
        return
    comm.all_reduce(stats[_G_MAX].view(torch.float32), "max")
    comm.all_reduce(stats[_COUNTS].view(torch.int64), "sum")


def reduce_n_out(stats: torch.Tensor, comm) -> None:
    """After phase_quantize: n_out <- sum over ranks (n and n_nonfinite are already global)."""
    if comm is None:
        return
    comm.all_reduce(stats[24:32].view(torch.int64), "sum")


def check_acc_range(desc, images_total: int, bits_g: int, bits_x: int) -> None:
    """The summed wgrad accumulator must fit int32 for the WHOLE batch, not only for one shard."""
    worst = images_total * desc.P * desc.Q * (1 << (bits_g - 1)) * ((1 << bits_x) - 1)
    if worst >= 1 << 31:
        raise lbt.LbtError(lbt.ERR_ACC_RANGE, "sharded wgrad")


def phase_stats(dY, state, stats, stream=None):
    lbt.grad_stats(dY, state, stats, stream=stream)


def phase_quantize(dY, index_offset, state, stats, q_dY, stream=None):
    lbt.quantize_grad_shard(dY, index_offset, state, stats, q_dY, stream=stream)


def phase_contract(desc, q_dY, q_W, q_X, scale_w, scale_x, state, stats, dX, dW, accW, bits_g, ws,
                   bits_w=4, bits_x=4, stream=None):
    lbt.update_interval(state, stats, stream=stream)
    lbt.qconv_dgrad_wgrad(desc, q_dY, q_W, q_X, lbt.stats_field_ptr(stats, "scale"), scale_w, scale_x,
                          dX, dW, None, accW, bits_g, bits_w, bits_x, ws,
                          dev_status=state[_DEV_STATUS], stream=stream)


def phase_finalize(accW, stats, scale_x, dW, stream=None):
    lbt.dequantize_acc(accW, lbt.stats_field_ptr(stats, "scale"), scale_x, dW, stream=stream)


def sharded_backward(desc, dY, q_W, q_X, scale_w, scale_x, state, stats, q_dY, dX, dW, accW, bits_g, ws,
                     index_offset: int, images_total: int, comm, bits_w=4, bits_x=4, stream=None):
    """One rank's part of the layer's backward pass.  `desc` describes the rank's slice (N = its
    images); `index_offset` is the slice's first gradient in the whole tensor (see shard_offsets);
    `images_total` the batch over all ranks.  On return dX holds the slice's input gradient, dW / accW
    the whole layer's weight gradient, `state` the updated clipping factor, `stats` the whole layer's
    statistics -- all identical to what one GPU computes on the whole batch."""
    check_acc_range(desc, images_total, bits_g, bits_x)
    # kernels and collectives on ONE stream: the collectives take torch's current stream
    scope = torch.cuda.stream(stream) if stream is not None else contextlib.nullcontext()
    with scope:
        phase_stats(dY, state, stats, stream)
        reduce_stats(stats, comm)
        phase_quantize(dY, index_offset, state, stats, q_dY, stream)
        reduce_n_out(stats, comm)
        phase_contract(desc, q_dY, q_W, q_X, scale_w, scale_x, state, stats, dX, dW, accW, bits_g, ws,
                       bits_w, bits_x, stream)
        if comm is not None:
            comm.all_reduce(accW, "sum")
            phase_finalize(accW, stats, scale_x, dW, stream)
