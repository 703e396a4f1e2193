"""ctypes binding of the C-ABI CUDA library (include/lbt.h): argument marshalling only.

Functions carry the names of the C entry points without the `lbt_` prefix.  Tensors are
torch CUDA tensors (used for device memory and streams only); every step of the path runs
in the library's kernels.  A missing library is an error: there is no other implementation.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblbt.so")

OK = 0
ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_UNSUPPORTED_BITS, ERR_ACC_RANGE = -1, -2, -3, -4
ERR_WORKSPACE, ERR_CUDA, ERR_NONFINITE, ERR_TIMEOUT, ERR_UNSUPPORTED = -5, -6, -7, -8, -9
ERR_SCRATCH_LIMIT = -10
ERR_BITS_MISMATCH = -11
STATIC_SCRATCH_BYTES = 8 << 20
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
OP_GRAD_STATS, OP_QUANTIZE, OP_GEMM_DGRAD, OP_GEMM_WGRAD, OP_CONV_BACKWARD, OP_GEMM_FORWARD, OP_CONV_FORWARD = range(7)

EXPORTS = (
    "lbt_workspace_bytes", "lbt_grad_stats", "lbt_quantize_grad", "lbt_update_interval",
    "lbt_qgemm_dgrad", "lbt_qgemm_wgrad", "lbt_qgemm_dgrad_static", "lbt_qconv_dgrad_wgrad", "lbt_qconv_backward",
    "lbt_qconv_backward_ex",
    "lbt_quantize_weight", "lbt_quantize_act", "lbt_qgemm_forward", "lbt_qconv_forward",
    "lbt_quantize_grad_shard", "lbt_dequantize_acc", "lbt_quantize_grad_fused",
    "lbt_grad_diagnostics", "lbt_diagnostics_workspace_bytes",
    "lbt_set_timing_events", "lbt_selftest_wait_timeout", "lbt_selftest_barrier_timeout", "lbt_status_string",
)
TIME_STATS, TIME_QUANTIZE, TIME_EXPAND, TIME_DGRAD, TIME_WGRAD, TIME_FORWARD, TIME_FWD_QUANT = range(7)


class IntervalState(C.Structure):
    """Mirror of `lbt_interval_state` (56 bytes)."""
    _fields_ = [("gamma", C.c_float), ("alpha", C.c_float), ("beta", C.c_float),
                ("gamma_min", C.c_float), ("gamma_max", C.c_float), ("bits", C.c_int32),
                ("rounding", C.c_uint32), ("reserved", C.c_uint32), ("seed", C.c_uint64),
                ("iter", C.c_uint64), ("dev_status", C.c_int32), ("reserved2", C.c_int32)]


class GradStats(C.Structure):
    """Mirror of `lbt_grad_stats_t` (40 bytes)."""
    _fields_ = [("g_max", C.c_float), ("c", C.c_float), ("scale", C.c_float),
                ("reserved", C.c_uint32), ("n", C.c_uint64), ("n_out", C.c_uint64),
                ("n_nonfinite", C.c_uint64)]


class GradDiag(C.Structure):
    """Mirror of `lbt_grad_diag_t` (88 bytes)."""
    _fields_ = [("n", C.c_uint64), ("n_large", C.c_uint64), ("n_in", C.c_uint64), ("n_out", C.c_uint64),
                ("sum_all", C.c_double), ("sum_large_in", C.c_double), ("sum_large_out", C.c_double),
                ("e_all", C.c_double), ("e_large", C.c_double), ("u_large", C.c_double),
                ("threshold", C.c_float), ("reserved", C.c_uint32)]


class GemmDesc(C.Structure):
    _fields_ = [("M", C.c_int64), ("O", C.c_int64), ("I", C.c_int64)]


class ConvDesc(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("N", "C", "H", "W", "K", "R", "S", "stride", "pad")]

    @property
    def P(self):
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Q(self):
        return (self.W + 2 * self.pad - self.S) // self.stride + 1


assert C.sizeof(IntervalState) == 56 and C.sizeof(GradStats) == 40

_lib = None


class LbtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def lib() -> C.CDLL:
    """Load liblbt.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2407_12637_b200.build` "
                "(there is no fallback implementation)")
        l = C.CDLL(LIB_PATH)
        vp, u64, sz, i64, i32 = C.c_void_p, C.c_uint64, C.c_size_t, C.c_int64, C.c_int
        l.lbt_workspace_bytes.restype = sz
        l.lbt_workspace_bytes.argtypes = [i32, vp]
        l.lbt_grad_stats.argtypes = [vp, u64, vp, vp, vp, sz, vp]
        l.lbt_quantize_grad.argtypes = [vp, u64, vp, vp, vp, vp, sz, vp]
        l.lbt_update_interval.argtypes = [vp, vp, vp]
        l.lbt_quantize_grad_shard.argtypes = [vp, u64, u64, vp, vp, vp, vp]
        l.lbt_dequantize_acc.argtypes = [vp, u64, vp, vp, vp, vp]
        l.lbt_quantize_grad_fused.argtypes = [vp, u64, vp, vp, vp, vp]
        l.lbt_grad_diagnostics.argtypes = [vp, u64, vp, i32, C.c_float, vp, vp, vp, sz, vp]
        l.lbt_diagnostics_workspace_bytes.argtypes = []
        for f in (l.lbt_quantize_weight, l.lbt_quantize_act):
            f.argtypes = [vp, u64, vp, i32, vp, vp, vp]
        l.lbt_qconv_forward.argtypes = [vp] * 7 + [i32, i32, vp, vp, sz, vp]
        for f in (l.lbt_qgemm_dgrad, l.lbt_qgemm_wgrad, l.lbt_qgemm_forward):
            f.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, vp, sz, vp]
        l.lbt_qgemm_dgrad_static.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, vp]
        l.lbt_qconv_dgrad_wgrad.argtypes = [vp] * 11 + [i32, i32, i32, vp, vp, sz, vp]
        l.lbt_qconv_backward.argtypes = [vp] * 13 + [i32, vp, sz, vp]
        l.lbt_qconv_backward_ex.argtypes = [vp] * 13 + [i32, vp, sz, i32, vp, vp]
        l.lbt_set_timing_events.argtypes = [i32, vp, vp]
        l.lbt_selftest_wait_timeout.argtypes = [vp, C.c_uint32, vp]
        l.lbt_selftest_barrier_timeout.argtypes = [vp, C.c_uint32, vp]
        for name in EXPORTS:
            if name not in ("lbt_workspace_bytes", "lbt_status_string", "lbt_diagnostics_workspace_bytes"):
                getattr(l, name).restype = C.c_int32
        l.lbt_diagnostics_workspace_bytes.restype = sz
        l.lbt_status_string.restype = C.c_char_p
        l.lbt_status_string.argtypes = [C.c_int32]
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().lbt_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise LbtError(status, where)


def _p(t) -> int:
    if t is None:
        return 0
    assert t.is_cuda and t.is_contiguous(), "device pointers come from contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream=None) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


# ------------------------------------------------------------------ device-resident structs
def new_state(gamma=1.0, alpha=1e-3, beta=1e-3, gamma_min=None, gamma_max=1.0, bits=4,
              rounding=ROUND_STOCHASTIC, seed=0, it=0, device="cuda") -> torch.Tensor:
    """A device `lbt_interval_state` as a 56-byte uint8 tensor."""
    s = IntervalState(gamma, alpha, beta, beta if gamma_min is None else gamma_min, gamma_max,
                      bits, rounding, 0, seed, it, 0, 0)
    return torch.frombuffer(bytearray(bytes(s)), dtype=torch.uint8).to(device)


def read_state(t: torch.Tensor) -> IntervalState:
    return IntervalState.from_buffer_copy(t.cpu().numpy().tobytes())


def new_stats(device="cuda") -> torch.Tensor:
    return torch.zeros(C.sizeof(GradStats), dtype=torch.uint8, device=device)


def read_stats(t: torch.Tensor) -> GradStats:
    return GradStats.from_buffer_copy(t.cpu().numpy().tobytes())


def stats_field_ptr(stats: torch.Tensor, name: str) -> int:
    """Device address of one field of a stats struct (e.g. 'scale' as a scale pointer)."""
    return stats.data_ptr() + getattr(GradStats, name).offset


_cudart = None


def _rt() -> C.CDLL:
    """The CUDA runtime torch has already loaded (events are plain driver handles, so events
    made here can be recorded by the library on any stream of the process)."""
    global _cudart
    if _cudart is None:
        torch.cuda.init()
        _cudart = C.CDLL("libcudart.so.12")
        _cudart.cudaEventCreate.argtypes = [C.POINTER(C.c_void_p)]
        _cudart.cudaEventDestroy.argtypes = [C.c_void_p]
        _cudart.cudaEventElapsedTime.argtypes = [C.POINTER(C.c_float), C.c_void_p, C.c_void_p]
    return _cudart


class TimingTap:
    """A pair of CUDA events the library records around every launch of one kernel class
    (`lbt_set_timing_events`).  `ms()` is valid after the stream has been synchronised."""

    def __init__(self, kernel_class: int):
        self.kernel_class = kernel_class
        self.start, self.stop = C.c_void_p(), C.c_void_p()
        for ev in (self.start, self.stop):
            if _rt().cudaEventCreate(C.byref(ev)) != 0:
                raise RuntimeError("cudaEventCreate failed")

    def arm(self):
        _check(lib().lbt_set_timing_events(self.kernel_class, self.start, self.stop),
               "lbt_set_timing_events")

    def disarm(self):
        _check(lib().lbt_set_timing_events(self.kernel_class, None, None), "lbt_set_timing_events")

    def ms(self) -> float:
        out = C.c_float()
        rc = _rt().cudaEventElapsedTime(C.byref(out), self.start, self.stop)
        if rc != 0:
            raise RuntimeError(f"cudaEventElapsedTime failed ({rc})")
        return out.value

    def close(self):
        for ev in (self.start, self.stop):
            _rt().cudaEventDestroy(ev)


# ------------------------------------------------------------------ entry points
def workspace_bytes(op: int, desc=None) -> int:
    return int(lib().lbt_workspace_bytes(op, C.byref(desc) if desc is not None else None))


def grad_stats(dY, state, stats, stream=None):
    _check(lib().lbt_grad_stats(_p(dY), dY.numel(), _p(state), _p(stats), None, 0,
                                _stream(stream)), "lbt_grad_stats")


def quantize_grad(dY, state, stats, q_out, stream=None):
    _check(lib().lbt_quantize_grad(_p(dY), dY.numel(), _p(state), _p(stats), _p(q_out), None, 0,
                                   _stream(stream)), "lbt_quantize_grad")


def update_interval(state, stats, stream=None):
    _check(lib().lbt_update_interval(_p(state), _p(stats), _stream(stream)), "lbt_update_interval")


def _ptr_or_tensor(x) -> int:
    return x if isinstance(x, int) else _p(x)


def qgemm_dgrad(q_dY, q_W, scale_g, scale_w, dX, acc_out, M, O, I, bits_g, bits_w, ws,
                dev_status=None, stream=None):
    _check(lib().lbt_qgemm_dgrad(_p(q_dY), _p(q_W), _ptr_or_tensor(scale_g), _ptr_or_tensor(scale_w),
                                 _p(dX), _p(acc_out), M, O, I, bits_g, bits_w, _p(dev_status),
                                 _p(ws), ws.numel() if ws is not None else 0, _stream(stream)),
           "lbt_qgemm_dgrad")


def selftest_wait_timeout(dev_status, limit_us: int, stream=None):
    """Run the kernels' bounded wait on a barrier nothing signals; *dev_status becomes ERR_TIMEOUT."""
    _check(lib().lbt_selftest_wait_timeout(_p(dev_status), int(limit_us), _stream(stream)),
           "lbt_selftest_wait_timeout")


def selftest_barrier_timeout(dev_status, limit_us: int, stream=None):
    """Run the one-launch quantizer's grid-barrier wait on a count that is never reached; *dev_status
    becomes ERR_TIMEOUT."""
    _check(lib().lbt_selftest_barrier_timeout(_p(dev_status), int(limit_us), _stream(stream)),
           "lbt_selftest_barrier_timeout")


def qgemm_dgrad_static(q_dY, q_W, scale_g, scale_w, dX, acc_out, M, O, I, bits_g, bits_w,
                       dev_status=None, stream=None):
    """`lbt_qgemm_dgrad` on the library's built-in scratch: for callers that may not allocate
    device memory.  Limited to problems whose workspace fits STATIC_SCRATCH_BYTES."""
    _check(lib().lbt_qgemm_dgrad_static(_p(q_dY), _p(q_W), _ptr_or_tensor(scale_g), _ptr_or_tensor(scale_w),
                                        _p(dX), _p(acc_out), M, O, I, bits_g, bits_w, _p(dev_status),
                                        _stream(stream)), "lbt_qgemm_dgrad_static")


def qgemm_wgrad(q_dY, q_X, scale_g, scale_x, dW, acc_out, M, O, I, bits_g, bits_x, ws,
                dev_status=None, stream=None):
    _check(lib().lbt_qgemm_wgrad(_p(q_dY), _p(q_X), _ptr_or_tensor(scale_g), _ptr_or_tensor(scale_x),
                                 _p(dW), _p(acc_out), M, O, I, bits_g, bits_x, _p(dev_status),
                                 _p(ws), ws.numel() if ws is not None else 0, _stream(stream)),
           "lbt_qgemm_wgrad")


def quantize_grad_shard(dY, index_offset, state, stats, q_out, stream=None):
    """`quantize_grad` for a shard that starts at element `index_offset` of the whole tensor."""
    _check(lib().lbt_quantize_grad_shard(_p(dY), dY.numel(), int(index_offset), _p(state), _p(stats), _p(q_out),
                                         _stream(stream)), "lbt_quantize_grad_shard")


def quantize_grad_fused(dY, state, stats, q_out, stream=None):
    """Statistics, quantization and the clipping-factor update in one cooperative launch."""
    _check(lib().lbt_quantize_grad_fused(_p(dY), dY.numel(), _p(state), _p(stats), _p(q_out), _stream(stream)),
           "lbt_quantize_grad_fused")


def grad_diagnostics(dY, q_codes, bits, alpha, stats, ws=None, stream=None) -> "GradDiag":
    """E(G), E(G_L), U(G_L) and the clip ratios (Sec. 3.2-3.3) of one quantized gradient tensor; synchronises
    to read the 88-byte result back."""
    out = torch.zeros(C.sizeof(GradDiag), dtype=torch.uint8, device=dY.device)
    if ws is None:
        ws = torch.empty(lib().lbt_diagnostics_workspace_bytes(), dtype=torch.uint8, device=dY.device)
    _check(lib().lbt_grad_diagnostics(_p(dY), dY.numel(), _p(q_codes), bits, float(alpha), _p(stats), _p(out), _p(ws),
                                      ws.numel(), _stream(stream)), "lbt_grad_diagnostics")
    return GradDiag.from_buffer_copy(out.cpu().numpy().tobytes())


def dequantize_acc(acc, scale_a, scale_b, out, stream=None):
    """out = (float)acc * fl32(s_a * s_b): the contractions' epilogue on summed int32 accumulators."""
    _check(lib().lbt_dequantize_acc(_p(acc), acc.numel(), _ptr_or_tensor(scale_a), _ptr_or_tensor(scale_b),
                                    _p(out), _stream(stream)), "lbt_dequantize_acc")


def quantize_weight(w, clip, bits, q_out, scale_out, stream=None):
    """Eq. (2): signed codes of `bits` bits into q_out, the scale into scale_out (device float)."""
    _check(lib().lbt_quantize_weight(_p(w), w.numel(), _ptr_or_tensor(clip), bits, _p(q_out),
                                     _ptr_or_tensor(scale_out), _stream(stream)), "lbt_quantize_weight")


def quantize_act(x, clip, bits, q_out, scale_out, stream=None):
    """Eq. (3): unsigned codes of `bits` bits into q_out, the scale into scale_out (device float)."""
    _check(lib().lbt_quantize_act(_p(x), x.numel(), _ptr_or_tensor(clip), bits, _p(q_out),
                                  _ptr_or_tensor(scale_out), _stream(stream)), "lbt_quantize_act")


def qgemm_forward(q_X, q_W, scale_x, scale_w, Y, acc_out, M, O, I, bits_x, bits_w, ws,
                  dev_status=None, stream=None):
    _check(lib().lbt_qgemm_forward(_p(q_X), _p(q_W), _ptr_or_tensor(scale_x), _ptr_or_tensor(scale_w),
                                   _p(Y), _p(acc_out), M, O, I, bits_x, bits_w, _p(dev_status),
                                   _p(ws), ws.numel() if ws is not None else 0, _stream(stream)),
           "lbt_qgemm_forward")


def qconv_forward(desc, q_X, q_W, scale_x, scale_w, Y, acc_out, bits_x, bits_w, ws,
                  dev_status=None, stream=None):
    _check(lib().lbt_qconv_forward(C.addressof(desc), _p(q_X), _p(q_W), _ptr_or_tensor(scale_x),
                                   _ptr_or_tensor(scale_w), _p(Y), _p(acc_out), bits_x, bits_w,
                                   _p(dev_status), _p(ws), ws.numel() if ws is not None else 0,
                                   _stream(stream)), "lbt_qconv_forward")


def qconv_dgrad_wgrad(desc, q_dY, q_W, q_X, scale_g, scale_w, scale_x, dX, dW, accX, accW,
                      bits_g, bits_w, bits_x, ws, dev_status=None, stream=None):
    _check(lib().lbt_qconv_dgrad_wgrad(
        C.addressof(desc), _p(q_dY), _p(q_W), _p(q_X), _ptr_or_tensor(scale_g),
        _ptr_or_tensor(scale_w), _ptr_or_tensor(scale_x), _p(dX), _p(dW), _p(accX), _p(accW),
        bits_g, bits_w, bits_x, _p(dev_status), _p(ws), ws.numel() if ws is not None else 0,
        _stream(stream)), "lbt_qconv_dgrad_wgrad")


def qconv_backward(desc, dY, q_W, q_X, scale_w, scale_x, state, stats, q_dY_out, dX, dW, accX,
                   accW, bits_g, ws, stream=None):
    _check(lib().lbt_qconv_backward(
        C.addressof(desc), _p(dY), _p(q_W), _p(q_X), _ptr_or_tensor(scale_w),
        _ptr_or_tensor(scale_x), _p(state), _p(stats), _p(q_dY_out), _p(dX), _p(dW), _p(accX),
        _p(accW), bits_g, _p(ws), ws.numel() if ws is not None else 0, _stream(stream)),
        "lbt_qconv_backward")


def qconv_backward_ex(desc, dY, q_W, q_X, scale_w, scale_x, state, stats, q_dY_out, dX, dW, accX,
                      accW, bits_g, ws, dy_stats_ready=False, dx_stats=None, stream=None):
    """`qconv_backward` that can skip the abs-max pass (`stats` already holds this dY's statistics) and
    leave the statistics of dX in `dx_stats` for the layer that receives dX as its gradient."""
    _check(lib().lbt_qconv_backward_ex(
        C.addressof(desc), _p(dY), _p(q_W), _p(q_X), _ptr_or_tensor(scale_w),
        _ptr_or_tensor(scale_x), _p(state), _p(stats), _p(q_dY_out), _p(dX), _p(dW), _p(accX),
        _p(accW), bits_g, _p(ws), ws.numel() if ws is not None else 0, int(bool(dy_stats_ready)),
        _p(dx_stats), _stream(stream)), "lbt_qconv_backward_ex")
