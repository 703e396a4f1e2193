"""The C-ABI library loads and exports every symbol include/lbt.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2407_12637_b200 import build as lib_build
from paper_2407_12637_b200 import lbt

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lbt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lbt_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib_build.build()
    so = ctypes.CDLL(lbt.LIB_PATH)
    names = _declared()
    assert set(names) == set(lbt.EXPORTS)
    for name in names:
        assert hasattr(so, name), name


def test_struct_mirrors_match_the_header_sizes():
    assert ctypes.sizeof(lbt.IntervalState) == 56
    assert ctypes.sizeof(lbt.GradStats) == 40
    assert lbt.GradStats.scale.offset == 8 and lbt.GradStats.n_out.offset == 24
    assert lbt.IntervalState.seed.offset == 32 and lbt.IntervalState.dev_status.offset == 48


def test_host_only_entry_points():
    lib_build.build()
    assert lbt.status_string(0) == "LBT_OK"
    assert lbt.status_string(lbt.ERR_TIMEOUT) == "LBT_ERR_TIMEOUT"
    assert lbt.status_string(-12345) == "LBT_ERR_UNKNOWN"
    assert lbt.workspace_bytes(lbt.OP_GRAD_STATS) == 0
    d = lbt.GemmDesc(128, 256, 256)
    need = lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, d)
    # int8 copies of dY, W, X
    assert need >= 128 * 256 + 256 * 256 + 128 * 256
    assert lbt.workspace_bytes(lbt.OP_GEMM_WGRAD, d) >= need          # a split reduction adds partial-sum slabs
    assert lbt.workspace_bytes(lbt.OP_GEMM_DGRAD, lbt.GemmDesc(0, 1, 1)) == 0
    c = lbt.ConvDesc(N=2, C=16, H=8, W=8, K=16, R=3, S=3, stride=1, pad=1)
    assert lbt.workspace_bytes(lbt.OP_CONV_BACKWARD, c) > 2 * 9 * 9 * 16 * 2
