"""ctypes front end of the C oracle (TEST INFRASTRUCTURE, see oracle/__init__.py).

Every function takes and returns numpy arrays; all arithmetic happens in
`lbt_oracle.c`.  Citations are to arXiv 2407.12637.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_u64, _i64, _f32, _int = C.c_uint64, C.c_int64, C.c_float, C.c_int
_p = C.c_void_p


class _ConvShape(C.Structure):
    _fields_ = [(name, _i64) for name in
                ("N", "C", "H", "W", "K", "R", "S", "stride", "pad", "P", "Q")]


def _sig(name, restype, *argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = list(argtypes)
    return fn


_philox = _sig("ref_philox4x32_10", None, _p, _p, _p)
_rand16 = _sig("ref_rand16", C.c_uint32, _u64, _u64, _u64)
_grad_stats = _sig("ref_grad_stats", None, _p, _u64, C.POINTER(_f32), C.POINTER(_u64))
_clip_count = _sig("ref_clip_count", _u64, _p, _u64, _f32)
_quantize = _sig("ref_quantize_grad", None, _p, _u64, _f32, _f32, _int, _int, _u64, _u64, _u64,
                 _p, C.POINTER(_f32), C.POINTER(_f32), C.POINTER(_u64))
_dequantize = _sig("ref_dequantize", None, _p, _u64, _f32, _p)
_pack = _sig("ref_pack", None, _p, _u64, _int, _p)
_unpack4 = _sig("ref_unpack4", None, _p, _u64, _int, _p)
_update_sign = _sig("ref_update_sign", _int, _int, _f32, _u64, _u64)
_update = _sig("ref_update_interval", _f32, _f32, _f32, _f32, _f32, _f32, _int, _u64, _u64, _u64)
_quantize_weight = _sig("ref_quantize_weight", None, _p, _u64, _f32, _int, _p, C.POINTER(_f32))
_quantize_act = _sig("ref_quantize_act", None, _p, _u64, _f32, _int, _p, C.POINTER(_f32))
_gemm_range = {
    "forward": _sig("ref_gemm_forward_range", None, _p, _p, _i64, _i64, _i64, _i64, _i64, _p),
    "dgrad": _sig("ref_gemm_dgrad_range", None, _p, _p, _i64, _i64, _i64, _i64, _i64, _p),
    "wgrad": _sig("ref_gemm_wgrad_range", None, _p, _p, _i64, _i64, _i64, _i64, _i64, _p),
}
_gemm_list = {
    "forward": _sig("ref_gemm_forward_list", None, _p, _p, _i64, _i64, _i64, _p, _i64, _p),
    "dgrad": _sig("ref_gemm_dgrad_list", None, _p, _p, _i64, _i64, _i64, _p, _i64, _p),
    "wgrad": _sig("ref_gemm_wgrad_list", None, _p, _p, _i64, _i64, _i64, _p, _i64, _p),
}
_conv_range = {
    "forward": _sig("ref_conv_forward_range", None, C.POINTER(_ConvShape), _p, _p, _i64, _i64, _p),
    "dgrad": _sig("ref_conv_dgrad_range", None, C.POINTER(_ConvShape), _p, _p, _i64, _i64, _p),
    "wgrad": _sig("ref_conv_wgrad_range", None, C.POINTER(_ConvShape), _p, _p, _i64, _i64, _p),
}
_conv_list = {
    "forward": _sig("ref_conv_forward_list", None, C.POINTER(_ConvShape), _p, _p, _p, _i64, _p),
    "dgrad": _sig("ref_conv_dgrad_list", None, C.POINTER(_ConvShape), _p, _p, _p, _i64, _p),
    "wgrad": _sig("ref_conv_wgrad_list", None, C.POINTER(_ConvShape), _p, _p, _p, _i64, _p),
}
_epilogue = _sig("ref_epilogue", _i64, _p, _i64, _f32, _f32, _p)


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _as(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


# --------------------------------------------------------------------------- Philox
def philox4x32_10(ctr, key) -> np.ndarray:
    """One Philox4x32-10 block (Salmon et al., SC'11): 4 counter words, 2 key words -> 4 words."""
    c = _as(ctr, np.uint32)
    k = _as(key, np.uint32)
    out = np.empty(4, np.uint32)
    _philox(_ptr(c), _ptr(k), _ptr(out))
    return out


def rand16(seed: int, it: int, i: int) -> int:
    """The 16 random bits that stochastic rounding uses for element i of call (seed, it)."""
    return int(_rand16(seed, it, i))


# --------------------------------------------------------------------------- statistics
def grad_stats(dY: np.ndarray):
    """g_max = max|g| over the layer (Sec. 3.1) and the count of non-finite elements."""
    g = _as(dY, np.float32).ravel()
    gm, bad = _f32(), _u64()
    _grad_stats(_ptr(g), g.size, C.byref(gm), C.byref(bad))
    return np.float32(gm.value), int(bad.value)


def clip_count(dY: np.ndarray, c) -> int:
    """#{|g| > c}, the clip-out count of Sec. 3.3 / Algorithm 1."""
    g = _as(dY, np.float32).ravel()
    return int(_clip_count(_ptr(g), g.size, np.float32(c)))


# --------------------------------------------------------------------------- quantizer
@dataclasses.dataclass
class Quantized:
    codes: np.ndarray      # int8, one per element, in [-qmax, qmax]
    c: np.float32          # clipping value c_g = gamma * g_max
    scale: np.float32      # s = c_g / (2^(b-1) - 1), Eq. (2)
    n_out: int             # clip-out count of this quantization


def quantize_grad(dY, gamma, g_max, bits, rounding=0, seed=0, it=0, n_nonfinite=0) -> Quantized:
    """Eq. (1), (2), (4) with c_g = gamma * g_max; rounding 0 nearest-even, 1 stochastic."""
    g = _as(dY, np.float32).ravel()
    codes = np.empty(g.size, np.int8)
    c, s, n_out = _f32(), _f32(), _u64()
    _quantize(_ptr(g), g.size, np.float32(gamma), np.float32(g_max), int(bits), int(rounding),
              int(seed), int(it), int(n_nonfinite), _ptr(codes), C.byref(c), C.byref(s),
              C.byref(n_out))
    return Quantized(codes, np.float32(c.value), np.float32(s.value), int(n_out.value))


def dequantize(codes, scale) -> np.ndarray:
    """Q(g) = s * code, Eq. (4)."""
    q = _as(codes, np.int8).ravel()
    out = np.empty(q.size, np.float32)
    _dequantize(_ptr(q), q.size, np.float32(scale), _ptr(out))
    return out


def quantize_weight(w, c, bits):
    """Eq. (1), (2), (4): signed codes in [-qmax, qmax] (int8) and the scale s = c / qmax."""
    w = _as(w, np.float32).ravel()
    codes = np.empty(w.size, np.int8)
    s = _f32()
    _quantize_weight(_ptr(w), w.size, float(np.float32(c)), int(bits), _ptr(codes), C.byref(s))
    return codes, np.float32(s.value)


def quantize_act(x, c, bits):
    """Eq. (1), (3), (4): unsigned codes in [0, 2^b - 1] (uint8) and the scale s = c / (2^b - 1)."""
    x = _as(x, np.float32).ravel()
    codes = np.empty(x.size, np.uint8)
    s = _f32()
    _quantize_act(_ptr(x), x.size, float(np.float32(c)), int(bits), _ptr(codes), C.byref(s))
    return codes, np.float32(s.value)


def pack(codes, bits) -> np.ndarray:
    """Storage bytes: two nibbles per byte (low nibble first) for bits <= 4, else int8."""
    q = _as(codes, np.int8).ravel()
    out = np.zeros((q.size + 1) // 2 if bits <= 4 else q.size, np.uint8)
    _pack(_ptr(q), q.size, int(bits), _ptr(out))
    return out


def unpack4(packed, n, signed) -> np.ndarray:
    """Nibble bytes -> int16 codes (sign- or zero-extended)."""
    b = _as(packed, np.uint8).ravel()
    out = np.empty(n, np.int16)
    _unpack4(_ptr(b), n, int(bool(signed)), _ptr(out))
    return out


# --------------------------------------------------------------------------- interval update
def update_sign(bits, alpha, n, n_out) -> int:
    """sign(T) of Eq. (16), decided on n_out (2^b - 1) versus alpha N."""
    return int(_update_sign(int(bits), np.float32(alpha), int(n), int(n_out)))


def update_interval(gamma, alpha, beta, gamma_min, gamma_max, bits, n, n_out, n_nonfinite=0):
    """Eq. (15): gamma_i = gamma_{i-1} + beta sign(T), clamped to [gamma_min, gamma_max]."""
    return np.float32(_update(np.float32(gamma), np.float32(alpha), np.float32(beta),
                              np.float32(gamma_min), np.float32(gamma_max), int(bits),
                              int(n), int(n_out), int(n_nonfinite)))


# --------------------------------------------------------------------------- contractions
def _codes16(a) -> np.ndarray:
    return _as(a, np.int16)


def _run_ranges(fn, total, threads, out):
    """Evaluate fn(begin, end, out_ptr) over [0, total), optionally split over threads."""
    if threads <= 1 or total < threads:
        fn(0, total, _ptr(out))
        return
    bounds = np.linspace(0, total, threads + 1).astype(np.int64)
    with ThreadPoolExecutor(threads) as ex:
        futs = [ex.submit(fn, int(b), int(e), _ptr(out) + 8 * int(b))
                for b, e in zip(bounds[:-1], bounds[1:]) if e > b]
        for f in futs:
            f.result()


def _run_list(fn, ix, threads):
    """Evaluate fn(idx_ptr, count, out_ptr) over the listed outputs, optionally split over threads."""
    out = np.empty(ix.size, np.int64)
    if threads <= 1 or ix.size < 4 * threads:
        fn(_ptr(ix), ix.size, _ptr(out))
        return out
    bounds = np.linspace(0, ix.size, threads + 1).astype(np.int64)
    with ThreadPoolExecutor(threads) as ex:
        futs = [ex.submit(fn, _ptr(ix) + 8 * int(b), int(e - b), _ptr(out) + 8 * int(b))
                for b, e in zip(bounds[:-1], bounds[1:]) if e > b]
        for f in futs:
            f.result()
    return out


def gemm_backward(kind, qdY, other, M, O, I, idx=None, threads=1) -> np.ndarray:
    """Linear layer Y = X W^T.  kind 'dgrad': sum_o qdY[m,o] qW[o,i] -> [M,I];
    kind 'wgrad': sum_m qdY[m,o] qX[m,i] -> [O,I].  int64 accumulators; `idx`
    restricts the evaluation to the listed flat output indices."""
    a = _codes16(qdY).ravel()
    b = _codes16(other).ravel()
    assert a.size == M * O and b.size == (O * I if kind == "dgrad" else M * I)
    total = (M if kind == "dgrad" else O) * I
    if idx is not None:
        ix = _as(idx, np.int64).ravel()
        return _run_list(lambda p, cnt, o: _gemm_list[kind](_ptr(a), _ptr(b), M, O, I, p, cnt, o), ix, threads)
    out = np.empty(total, np.int64)
    _run_ranges(lambda b0, e0, p: _gemm_range[kind](_ptr(a), _ptr(b), M, O, I, b0, e0, p),
                total, threads, out)
    return out.reshape((M if kind == "dgrad" else O), I)


def gemm_forward(qX, qW, M, O, I, idx=None, threads=1) -> np.ndarray:
    """Linear layer on codes: accY[m,o] = sum_i qX[m,i] qW[o,i] -> [M,O], int64."""
    a = _codes16(qX).ravel()
    b = _codes16(qW).ravel()
    assert a.size == M * I and b.size == O * I
    if idx is not None:
        ix = _as(idx, np.int64).ravel()
        return _run_list(lambda p, cnt, o: _gemm_list["forward"](_ptr(a), _ptr(b), M, O, I, p, cnt, o), ix, threads)
    out = np.empty(M * O, np.int64)
    _run_ranges(lambda b0, e0, p: _gemm_range["forward"](_ptr(a), _ptr(b), M, O, I, b0, e0, p),
                M * O, threads, out)
    return out.reshape(M, O)


@dataclasses.dataclass(frozen=True)
class ConvShape:
    """NHWC activations, KRSC weights; Y[n,p,q,k] = sum X[n,p*st+r-pad,q*st+s-pad,c] W[k,r,s,c]."""
    N: int
    C: int
    H: int
    W: int
    K: int
    R: int
    S: int
    stride: int = 1
    pad: int = 0

    @property
    def P(self):
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Q(self):
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    def _c(self):
        return _ConvShape(self.N, self.C, self.H, self.W, self.K, self.R, self.S,
                          self.stride, self.pad, self.P, self.Q)


def conv_backward(kind, d: ConvShape, qdY, other, idx=None, threads=1) -> np.ndarray:
    """kind 'dgrad': accX[n,h,w,c] from qdY[N,P,Q,K] and qW[K,R,S,C];
    kind 'wgrad': accW[k,r,s,c] from qdY and qX[N,H,W,C].  int64 accumulators."""
    a = _codes16(qdY).ravel()
    b = _codes16(other).ravel()
    assert a.size == d.N * d.P * d.Q * d.K
    if kind == "dgrad":
        assert b.size == d.K * d.R * d.S * d.C
        shape = (d.N, d.H, d.W, d.C)
    else:
        assert b.size == d.N * d.H * d.W * d.C
        shape = (d.K, d.R, d.S, d.C)
    cs = d._c()
    if idx is not None:
        ix = _as(idx, np.int64).ravel()
        return _run_list(lambda p, cnt, o: _conv_list[kind](C.byref(cs), _ptr(a), _ptr(b), p, cnt, o), ix, threads)
    total = int(np.prod(shape))
    out = np.empty(total, np.int64)
    _run_ranges(lambda b0, e0, p: _conv_range[kind](C.byref(cs), _ptr(a), _ptr(b), b0, e0, p),
                total, threads, out)
    return out.reshape(shape)


def conv_forward(d: ConvShape, qX, qW, idx=None, threads=1) -> np.ndarray:
    """accY[n,p,q,k] from qX[N,H,W,C] and qW[K,R,S,C]; int64 accumulators."""
    a = _codes16(qX).ravel()
    b = _codes16(qW).ravel()
    assert a.size == d.N * d.H * d.W * d.C and b.size == d.K * d.R * d.S * d.C
    shape = (d.N, d.P, d.Q, d.K)
    cs = d._c()
    if idx is not None:
        ix = _as(idx, np.int64).ravel()
        return _run_list(lambda p, cnt, o: _conv_list["forward"](C.byref(cs), _ptr(a), _ptr(b), p, cnt, o), ix, threads)
    total = int(np.prod(shape))
    out = np.empty(total, np.int64)
    _run_ranges(lambda b0, e0, p: _conv_range["forward"](C.byref(cs), _ptr(a), _ptr(b), b0, e0, p),
                total, threads, out)
    return out.reshape(shape)


def epilogue(acc, s_a, s_b):
    """fp32 output (float)acc * fl32(s_a * s_b); also the count of accumulators outside int32."""
    a = _as(acc, np.int64)
    out = np.empty(a.size, np.float32)
    over = _epilogue(_ptr(a.ravel()), a.size, np.float32(s_a), np.float32(s_b), _ptr(out))
    return out.reshape(a.shape), int(over)
