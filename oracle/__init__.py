"""ctypes front end of the CPU oracle (oracle/hq_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU
baseline leg of bench.py.  The product package never imports this module.

Each wrapper only marshals numpy arrays; all arithmetic is in hq_oracle.cpp.  The
`Layer` helper strings the oracle's steps together in the order of Sec. 4 / 4.1 of the
paper: accumulate, take min/max at the accumulator, quantize with the range of the
previous iteration, then update the range (iteration 0 runs the dynamic path, Eq. 1).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hq_oracle.cpp")
_LIB = os.path.join(_HERE, "libhq_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fused multiply-add, OpenMP over output rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class Range(C.Structure):
    _fields_ = [("q_min", C.c_float), ("q_max", C.c_float), ("scale", C.c_float), ("inv_scale", C.c_float),
                ("zero_point", C.c_int32), ("step", C.c_uint32)]

    def copy(self) -> "Range":
        return Range(self.q_min, self.q_max, self.scale, self.inv_scale, self.zero_point, self.step)

    def astuple(self):
        return (self.q_min, self.q_max, self.scale, self.inv_scale, self.zero_point, self.step)


class Conv(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("N", "H", "W", "C", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w", "groups")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i8p, i32p, i64p, f32p = (C.POINTER(t) for t in (C.c_int8, C.c_int32, C.c_int64, C.c_float))
        rp, cp = C.POINTER(Range), C.POINTER(Conv)
        L.hqo_out_h.argtypes = [cp]; L.hqo_out_h.restype = C.c_int32
        L.hqo_out_w.argtypes = [cp]; L.hqo_out_w.restype = C.c_int32
        L.hqo_derive.argtypes = [rp]; L.hqo_derive.restype = None
        L.hqo_linear_acc.argtypes = [C.c_int, C.c_int, C.c_int, i8p, C.c_int, i8p, C.c_int, i32p, i32p]; L.hqo_linear_acc.restype = C.c_int
        L.hqo_linear_wgrad_acc.argtypes = [C.c_int, C.c_int, C.c_int, i8p, C.c_int, i8p, C.c_int, i32p]; L.hqo_linear_wgrad_acc.restype = C.c_int
        L.hqo_conv_wgrad_acc.argtypes = [cp, i8p, C.c_int, i8p, C.c_int, i32p]; L.hqo_conv_wgrad_acc.restype = C.c_int
        L.hqo_scale_to_real.argtypes = [i32p, C.c_int64, C.c_float, f32p]; L.hqo_scale_to_real.restype = None
        L.hqo_conv_fwd_acc.argtypes = [cp, i8p, C.c_int, i8p, C.c_int, i32p]; L.hqo_conv_fwd_acc.restype = C.c_int
        L.hqo_conv_bwd_data_acc.argtypes = [cp, i8p, C.c_int, i8p, C.c_int, i32p]; L.hqo_conv_bwd_data_acc.restype = C.c_int
        L.hqo_linear_acc_at.argtypes = [C.c_int, C.c_int, C.c_int, i8p, C.c_int, i8p, C.c_int, i32p, i64p, C.c_int64, i64p]; L.hqo_linear_acc_at.restype = None
        L.hqo_conv_fwd_acc_at.argtypes = [cp, i8p, C.c_int, i8p, C.c_int, i64p, C.c_int64, i64p]; L.hqo_conv_fwd_acc_at.restype = None
        L.hqo_conv_bwd_data_acc_at.argtypes = [cp, i8p, C.c_int, i8p, C.c_int, i64p, C.c_int64, i64p]; L.hqo_conv_bwd_data_acc_at.restype = None
        L.hqo_minmax.argtypes = [i32p, C.c_int64, i32p, i32p]; L.hqo_minmax.restype = None
        L.hqo_quantize.argtypes = [i32p, C.c_int64, C.c_float, rp, i8p]; L.hqo_quantize.restype = None
        L.hqo_saturation.argtypes = [i32p, C.c_int64, C.c_float, rp, C.c_int, C.c_uint32, C.c_uint32, C.c_int64, i64p, i64p]; L.hqo_saturation.restype = None
        L.hqo_range_update.argtypes = [rp, C.c_int32, C.c_int32, C.c_float, C.c_float]; L.hqo_range_update.restype = None
        L.hqo_dynamic.argtypes = [i32p, C.c_int64, C.c_float, rp, f32p, i8p]; L.hqo_dynamic.restype = None
        L.hqo_acc_scale.argtypes = [C.c_float, C.c_float]; L.hqo_acc_scale.restype = C.c_float
        L.hqo_dequant.argtypes = [C.c_int8, rp]; L.hqo_dequant.restype = C.c_float
        _lib = L
    return _lib


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(C.POINTER(t))


def _i8(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.int8
    return a


def conv_desc(N, H, W, Cin, K, R, S, stride=1, pad=0, groups=1) -> Conv:
    sh, sw = (stride, stride) if np.isscalar(stride) else stride
    ph, pw = (pad, pad) if np.isscalar(pad) else pad
    return Conv(N, H, W, Cin, K, R, S, sh, sw, ph, pw, groups)


def out_hw(d: Conv):
    return lib().hqo_out_h(C.byref(d)), lib().hqo_out_w(C.byref(d))


def derive(q: Range) -> Range:
    lib().hqo_derive(C.byref(q))
    return q


def linear_acc(X, zx, W, zw=0, bias=None) -> np.ndarray:
    X, W = _i8(X), _i8(W)
    M, K = X.shape
    N = W.shape[0]
    assert W.shape[1] == K
    acc = np.empty((M, N), np.int32)
    b = None if bias is None else _p(np.ascontiguousarray(bias, dtype=np.int32), C.c_int32)
    ovf = lib().hqo_linear_acc(M, N, K, _p(X, C.c_int8), int(zx), _p(W, C.c_int8), int(zw), b, _p(acc, C.c_int32))
    assert ovf == 0, "int32 accumulator overflow"
    return acc


def linear_wgrad_acc(dY, zdy, X, zx) -> np.ndarray:
    """int32 g[n,k] = sum_m (dy[m,n] - z_dy) * (x[m,k] - z_x): the weight gradient of a linear layer in accumulator units."""
    dY, X = _i8(dY), _i8(X)
    M, N = dY.shape
    K = X.shape[1]
    assert X.shape[0] == M
    g = np.empty((N, K), np.int32)
    ovf = lib().hqo_linear_wgrad_acc(M, N, K, _p(dY, C.c_int8), int(zdy), _p(X, C.c_int8), int(zx), _p(g, C.c_int32))
    assert ovf == 0, "int32 accumulator overflow"
    return g


def conv_wgrad_acc(d: Conv, dY, zdy, X, zx) -> np.ndarray:
    """int32 g[k,r,s,c] = sum over output pixels of (dy - z_dy) * (x - z_x), padded taps skipped; depthwise: g[c,r,s]."""
    assert d.groups == 1 or (d.groups == d.C and d.K == d.C)
    dY, X = _i8(dY), _i8(X)
    Ho, Wo = out_hw(d)
    assert dY.shape == (d.N, Ho, Wo, d.K) and X.shape == (d.N, d.H, d.W, d.C)
    g = np.empty((d.K, d.R, d.S, d.C) if d.groups == 1 else (d.C, d.R, d.S), np.int32)
    ovf = lib().hqo_conv_wgrad_acc(C.byref(d), _p(dY, C.c_int8), int(zdy), _p(X, C.c_int8), int(zx), _p(g, C.c_int32))
    assert ovf == 0, "int32 accumulator overflow"
    return g


def scale_to_real(acc: np.ndarray, s_acc: float) -> np.ndarray:
    """fl(float(acc) * s_acc) per element, in binary32 (the weight gradient is kept in FP32)."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    out = np.empty(acc.shape, np.float32)
    lib().hqo_scale_to_real(_p(acc, C.c_int32), acc.size, C.c_float(s_acc), _p(out, C.c_float))
    return out


def conv_fwd_acc(d: Conv, X, zx, W, zw=0) -> np.ndarray:
    X, W = _i8(X), _i8(W)
    Ho, Wo = out_hw(d)
    acc = np.empty((d.N, Ho, Wo, d.K), np.int32)
    ovf = lib().hqo_conv_fwd_acc(C.byref(d), _p(X, C.c_int8), int(zx), _p(W, C.c_int8), int(zw), _p(acc, C.c_int32))
    assert ovf == 0, "int32 accumulator overflow"
    return acc


def conv_bwd_data_acc(d: Conv, dY, zdy, W, zw=0) -> np.ndarray:
    dY, W = _i8(dY), _i8(W)
    acc = np.empty((d.N, d.H, d.W, d.C), np.int32)
    ovf = lib().hqo_conv_bwd_data_acc(C.byref(d), _p(dY, C.c_int8), int(zdy), _p(W, C.c_int8), int(zw), _p(acc, C.c_int32))
    assert ovf == 0, "int32 accumulator overflow"
    return acc


def linear_acc_at(X, zx, W, idx, zw=0, bias=None) -> np.ndarray:
    X, W = _i8(X), _i8(W)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    out = np.empty(idx.shape, np.int64)
    b = None if bias is None else _p(np.ascontiguousarray(bias, dtype=np.int32), C.c_int32)
    lib().hqo_linear_acc_at(X.shape[0], W.shape[0], X.shape[1], _p(X, C.c_int8), int(zx), _p(W, C.c_int8), int(zw), b, _p(idx, C.c_int64), idx.size, _p(out, C.c_int64))
    return out


def conv_fwd_acc_at(d: Conv, X, zx, W, idx, zw=0) -> np.ndarray:
    X, W = _i8(X), _i8(W)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    out = np.empty(idx.shape, np.int64)
    lib().hqo_conv_fwd_acc_at(C.byref(d), _p(X, C.c_int8), int(zx), _p(W, C.c_int8), int(zw), _p(idx, C.c_int64), idx.size, _p(out, C.c_int64))
    return out


def conv_bwd_data_acc_at(d: Conv, dY, zdy, W, idx, zw=0) -> np.ndarray:
    dY, W = _i8(dY), _i8(W)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    out = np.empty(idx.shape, np.int64)
    lib().hqo_conv_bwd_data_acc_at(C.byref(d), _p(dY, C.c_int8), int(zdy), _p(W, C.c_int8), int(zw), _p(idx, C.c_int64), idx.size, _p(out, C.c_int64))
    return out


def minmax(acc: np.ndarray):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    mn, mx = C.c_int32(), C.c_int32()
    lib().hqo_minmax(_p(acc, C.c_int32), acc.size, C.byref(mn), C.byref(mx))
    return mn.value, mx.value


def quantize(acc: np.ndarray, s_acc: float, q: Range) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    out = np.empty(acc.shape, np.int8)
    lib().hqo_quantize(_p(acc, C.c_int32), acc.size, C.c_float(s_acc), C.byref(q), _p(out, C.c_int8))
    return out


def saturation(acc: np.ndarray, s_acc: float, q: Range, sr_seed: int | None = None, iteration: int = 0, first: int = 0):
    """(below, above): how many outputs the quantizer clips to the lowest / highest level (rounded grid coordinate + zero
    point outside -128..127).  sr_seed: None = round half to even, else stochastic rounding with that seed and iteration."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    b, a = C.c_int64(), C.c_int64()
    lib().hqo_saturation(_p(acc, C.c_int32), acc.size, C.c_float(s_acc), C.byref(q), 0 if sr_seed is None else 1,
                         C.c_uint32(0 if sr_seed is None else sr_seed), C.c_uint32(iteration), C.c_int64(first), C.byref(b), C.byref(a))
    return b.value, a.value


def range_update(q: Range, mn: int, mx: int, s_acc: float, eta: float) -> Range:
    lib().hqo_range_update(C.byref(q), int(mn), int(mx), C.c_float(s_acc), C.c_float(eta))
    return q


def dynamic(acc: np.ndarray, s_acc: float, q: Range):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    yf = np.empty(acc.shape, np.float32)
    out = np.empty(acc.shape, np.int8)
    lib().hqo_dynamic(_p(acc, C.c_int32), acc.size, C.c_float(s_acc), C.byref(q), _p(yf, C.c_float), _p(out, C.c_int8))
    return yf, out


def philox4x32_10(counter, key):
    """Four 32-bit words of Philox4x32-10 for a 4-word counter and a 2-word key."""
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in counter])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    out = (C.c_uint32 * 4)()
    lib().hqo_philox4x32_10(c, k, out)
    return [int(x) for x in out]


def draw16(seed: int, iteration: int, e: int) -> int:
    """The 16-bit draw of the output element with linear index e."""
    lib().hqo_draw16.restype = C.c_uint32
    return int(lib().hqo_draw16(C.c_uint32(seed), C.c_uint32(iteration), C.c_int64(e)))


def quantize_sr(acc: np.ndarray, s_acc: float, q: Range, seed: int, iteration: int, first: int = 0) -> np.ndarray:
    """Static quantization with stochastic rounding; element i (C order) has linear index first + i."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    out = np.empty(acc.shape, np.int8)
    lib().hqo_quantize_sr(_p(acc, C.c_int32), C.c_int64(acc.size), C.c_float(s_acc), C.byref(q), C.c_uint32(seed), C.c_uint32(iteration),
                          C.c_int64(first), _p(out, C.c_int8))
    return out


def dynamic_sr(acc: np.ndarray, s_acc: float, q: Range, seed: int):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    yf = np.empty(acc.shape, np.float32)
    out = np.empty(acc.shape, np.int8)
    lib().hqo_dynamic_sr(_p(acc, C.c_int32), C.c_int64(acc.size), C.c_float(s_acc), C.byref(q), C.c_uint32(seed), _p(yf, C.c_float),
                         _p(out, C.c_int8))
    return yf, out


def dynamic_running(acc: np.ndarray, s_acc: float, q: Range, eta: float):
    """Running min-max: the dynamic path with the moving average of Eq. 2-3 taken over the current tensor's min/max."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    yf = np.empty(acc.shape, np.float32)
    out = np.empty(acc.shape, np.int8)
    lib().hqo_dynamic_running(_p(acc, C.c_int32), C.c_int64(acc.size), C.c_float(s_acc), C.byref(q), C.c_float(eta), _p(yf, C.c_float),
                              _p(out, C.c_int8))
    return yf, out


def acc_scale(s_x: float, s_w: float) -> float:
    return float(lib().hqo_acc_scale(C.c_float(s_x), C.c_float(s_w)))


def dequant(code: int, q: Range) -> float:
    return float(lib().hqo_dequant(C.c_int8(int(code)), C.byref(q)))


@dataclass
class StepResult:
    acc: np.ndarray
    mn: int
    mx: int
    s_acc: float
    q: np.ndarray          # int8 output
    mode: str              # "dynamic" (t = 0) or "hindsight"


class Layer:
    """One quantized tensor's life over iterations, in the paper's order.

    step(acc, s_acc): iteration 0 -> dynamic path (its own min/max, Eq. 1) which
    initialises the range; afterwards -> quantize with the range estimated on the
    previous iterations, then apply Eq. 2-3 with this tensor's min/max.
    """

    def __init__(self, eta: float = 0.9, sr_seed: int | None = None):
        """sr_seed: None = round to nearest even; an integer = stochastic rounding with that seed
        (the iteration number of the draws is the state's update count)."""
        self.eta = float(eta)
        self.state = Range()
        self.sr_seed = sr_seed

    def step(self, acc: np.ndarray, s_acc: float, force_state: Range | None = None) -> StepResult:
        if force_state is not None:
            self.state = force_state.copy()
        mn, mx = minmax(acc)
        if self.state.step == 0:
            if self.sr_seed is None:
                _, q = dynamic(acc, s_acc, self.state)
            else:
                _, q = dynamic_sr(acc, s_acc, self.state, self.sr_seed)
            return StepResult(acc, mn, mx, s_acc, q, "dynamic")
        if self.sr_seed is None:
            q = quantize(acc, s_acc, self.state)
        else:
            q = quantize_sr(acc, s_acc, self.state, self.sr_seed, self.state.step)
        range_update(self.state, mn, mx, s_acc, self.eta)
        return StepResult(acc, mn, mx, s_acc, q, "hindsight")
