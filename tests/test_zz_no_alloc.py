"""`lbt_qgemm_dgrad_static`: the dgrad contraction for callers that may not allocate device memory
(a layer living inside a framework that owns all of HBM, a loop that cannot afford the device stall
of cudaMalloc / cudaFree).  It must give exactly what `lbt_qgemm_dgrad` gives with a caller-supplied
workspace -- and what the CPU oracle gives -- and a call must leave the amount of allocated device
memory as it found it.  The file name makes pytest collect it last, after every other test."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, synth

pytestmark = pytest.mark.gpu


def _inputs(M, O, I, bits_g, seed):
    q_dY = synth.code_bytes_torch(M * O // 2 if bits_g <= 4 else M * O, seed, 0)
    q_W = synth.code_bytes_torch(O * I // 2, seed, 1)
    return q_dY, q_W


def _both(M, O, I, bits_g, seed):
    """Run the workspace entry point and the built-in-scratch entry point on the same inputs."""
    q_dY, q_W = _inputs(M, O, I, bits_g, seed)
    sc = torch.tensor([1.25e-4, 0.01], device="cuda")
    ws = torch.empty(lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, lbt.GemmDesc(M, O, I)), dtype=torch.uint8, device="cuda")
    out = {}
    for name in ("workspace", "static"):
        dX = torch.full((M, I), float("nan"), device="cuda")
        acc = torch.full((M, I), -77, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if name == "workspace":
            lbt.qgemm_dgrad(q_dY, q_W, sc.data_ptr(), sc.data_ptr() + 4, dX, acc, M, O, I, bits_g, 4, ws, status)
        else:
            lbt.qgemm_dgrad_static(q_dY, q_W, sc.data_ptr(), sc.data_ptr() + 4, dX, acc, M, O, I, bits_g, 4, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        out[name] = (dX.cpu().numpy(), acc.cpu().numpy())
    out["inputs"] = (q_dY, q_W)
    return out


def _assert_same(out):
    (dx_a, acc_a), (dx_b, acc_b) = out["workspace"], out["static"]
    assert np.array_equal(acc_a, acc_b)                       # int32 accumulators: bit for bit
    tol = 1e-6 * np.abs(dx_a) + 1e-6 * 1.25e-4 * 0.01         # the fp32 tolerance of the parity tests
    assert np.all(np.abs(dx_a - dx_b) <= tol)


def _assert_matches_oracle(out, M, O, I, bits_g):
    """The built-in-scratch result against the CPU oracle: accumulators bit for bit, fp32 within 1e-6."""
    q_dY, q_W = (t.cpu().numpy() for t in out["inputs"])
    c_dY = ref.unpack4(q_dY, M * O, True) if bits_g <= 4 else q_dY.view(np.int8).astype(np.int16)
    c_W = ref.unpack4(q_W, O * I, True)
    want = ref.gemm_backward("dgrad", c_dY, c_W, M, O, I, threads=8)
    dx, acc = out["static"]
    assert np.array_equal(acc, want.astype(np.int32))
    f, over = ref.epilogue(want, 1.25e-4, 0.01)
    assert over == 0
    assert np.all(np.abs(dx - f) <= 1e-6 * np.abs(f) + 1e-6 * 1.25e-4 * 0.01)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # a larger problem first, then a smaller one with other data: the second call must not be
    # disturbed by what the first left in the shared scratch
    first = _both(640, 384, 520, 4, seed=11)
    _assert_same(first)
    _assert_matches_oracle(first, 640, 384, 520, 4)
    second = _both(130, 72, 40, 8, seed=12)
    _assert_same(second)
    _assert_matches_oracle(second, 130, 72, 40, 8)


def test_a_call_allocates_no_device_memory_and_may_keep_its_status_in_the_scratch():
    """What the entry point is for: after a first call (which looks the scratch address up), further calls
    change neither torch's allocation count nor the free memory the driver reports.  Without a caller's
    status word (dev_status = NULL) the kernels' status lives inside the built-in scratch."""
    M, O, I = 384, 200, 264
    q_dY, q_W = _inputs(M, O, I, 4, 14)
    sc = torch.tensor([1.25e-4, 0.01], device="cuda")
    dX = torch.full((M, I), float("nan"), device="cuda")
    acc = torch.full((M, I), -77, dtype=torch.int32, device="cuda")
    args = (q_dY, q_W, sc.data_ptr(), sc.data_ptr() + 4, dX, acc, M, O, I, 4, 4)
    lbt.qgemm_dgrad_static(*args, None)                    # set-up call
    torch.cuda.synchronize()
    allocated, (free, _total) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
    for _ in range(3):
        lbt.qgemm_dgrad_static(*args, None)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == allocated
    assert torch.cuda.mem_get_info()[0] == free
    out = {"static": (dX.cpu().numpy(), acc.cpu().numpy()), "inputs": (q_dY, q_W)}
    _assert_matches_oracle(out, M, O, I, 4)


def test_problems_beyond_the_built_in_scratch_are_refused():
    M = O = I = 2048
    assert lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, lbt.GemmDesc(M, O, I)) > lbt.STATIC_SCRATCH_BYTES
    q_dY, q_W = _inputs(M, O, I, 4, 13)
    sc = torch.tensor([1.0, 1.0], device="cuda")
    dX = torch.zeros(M, I, device="cuda")
    rc = lbt.lib().lbt_qgemm_dgrad_static(q_dY.data_ptr(), q_W.data_ptr(), sc.data_ptr(), sc.data_ptr() + 4,
                                          dX.data_ptr(), None, M, O, I, 4, 4, None, 0)
    assert rc == lbt.ERR_SCRATCH_LIMIT
    assert lbt.status_string(rc) == "LBT_ERR_SCRATCH_LIMIT"
    assert lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, lbt.GemmDesc(1024, 1024, 1024)) <= lbt.STATIC_SCRATCH_BYTES
