"""A wait that nothing satisfies must end in LBT_ERR_TIMEOUT and leave the context usable: no trap, no
hang.  The wait routine under test is the one every mbarrier wait of the contraction kernels uses."""
import time

import numpy as np
import pytest
import torch

from paper_2407_12637_b200 import lbt, synth

pytestmark = pytest.mark.gpu


def test_lost_signal_becomes_a_status_code():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    lbt.selftest_wait_timeout(status, 200_000)          # 0.2 s
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert int(status.item()) == lbt.ERR_TIMEOUT
    assert 0.15 < waited < 5.0
    # sticky: a second expiry does not overwrite, and a pre-set code survives
    status.fill_(lbt.ERR_NONFINITE)
    lbt.selftest_wait_timeout(status, 1000)
    torch.cuda.synchronize()
    assert int(status.item()) == lbt.ERR_NONFINITE


def test_context_still_works_after_a_timeout():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lbt.selftest_wait_timeout(status, 1000)
    M, O, I = 256, 256, 256
    q_dY, q_W = synth.code_bytes_torch(M * O // 2, 1, 0), synth.code_bytes_torch(O * I // 2, 1, 1)
    sc = torch.tensor([1.0, 1.0], device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, lbt.GemmDesc(M, O, I)), dtype=torch.uint8, device="cuda")
    dX = torch.empty(M, I, device="cuda")
    ok = torch.zeros(1, dtype=torch.int32, device="cuda")
    lbt.qgemm_dgrad(q_dY, q_W, sc.data_ptr(), sc.data_ptr() + 4, dX, None, M, O, I, 4, 4, ws, ok)
    torch.cuda.synchronize()
    assert int(status.item()) == lbt.ERR_TIMEOUT and int(ok.item()) == 0
    assert np.isfinite(dX.cpu().numpy()).all()


def test_argument_checks():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    L = lbt.lib()
    assert L.lbt_selftest_wait_timeout(None, 10, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_selftest_wait_timeout(status.data_ptr(), 0, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_selftest_wait_timeout(status.data_ptr(), 2_000_000, 0) == lbt.ERR_INVALID_ARG


def test_grid_barrier_that_is_never_completed_gives_up():
    """The counter barrier of the one-launch quantizer: a block that waits for arrivals that never come
    records LBT_ERR_TIMEOUT after its limit, and the quantizer that uses the barrier still runs afterwards."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    lbt.selftest_barrier_timeout(status, 200_000)       # 0.2 s
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert int(status.item()) == lbt.ERR_TIMEOUT
    assert 0.15 < waited < 5.0
    # the context is usable and the real barrier completes: the one-launch quantizer runs clean
    n = 100_003
    g = synth.laplace_outliers(n, 1e-3, seed=3)
    st, stats = lbt.new_state(gamma=0.7, bits=4, seed=3), lbt.new_stats()
    q = torch.empty((n + 1) // 2, dtype=torch.uint8, device="cuda")
    lbt.quantize_grad_fused(torch.from_numpy(g).cuda(), st, stats, q)
    torch.cuda.synchronize()
    state = lbt.read_state(st)
    assert state.dev_status == 0 and state.iter == 1 and lbt.read_stats(stats).reserved == 0
    L = lbt.lib()
    assert L.lbt_selftest_barrier_timeout(None, 10, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_selftest_barrier_timeout(status.data_ptr(), 0, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_selftest_barrier_timeout(status.data_ptr(), 2_000_000, 0) == lbt.ERR_INVALID_ARG
