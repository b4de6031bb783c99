"""Python face of the C-ABI library libhq.so: the same call names as include/hq.h.

Argument marshalling only.  Tensors are passed as objects with a ``data_ptr()`` (torch
tensors) or as raw integer device addresses; streams as ``torch.cuda.Stream`` objects, raw
handles or None.  There is no fallback: if the compiled library is missing, the first call
raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhq.so")

HQ_OK = 0
STATUS_NAMES = {0: "HQ_OK", 1: "HQ_ERR_INVALID_ARG", 2: "HQ_ERR_UNSUPPORTED", 3: "HQ_ERR_ALIGNMENT", 4: "HQ_ERR_CUDA",
                5: "HQ_ERR_NOT_INITIALIZED", 6: "HQ_ERR_TIMEOUT"}
DIR_FWD, DIR_BWD_DATA = 0, 1
OP_LINEAR, OP_CONV_FWD, OP_CONV_BWD_DATA = 0, 1, 2

# every extern "C" symbol include/hq.h declares
EXPORTS = ["hq_create", "hq_destroy", "hq_status_string", "hq_last_error", "hq_get_async_error", "hq_launch_count", "hq_pair_launch_count",
           "hq_set_option",
           "hq_weights_prepare", "hq_weights_prepare_zp", "hq_linear_prepare", "hq_linear_fwd_prepared", "hq_weights_release", "hq_linear_fwd", "hq_conv_fwd", "hq_conv_bwd_data", "hq_range_update",
           "hq_dynamic_quant", "hq_dynamic_quant_static", "hq_debug_accumulate", "hq_linear_wgrad", "hq_conv_wgrad",
           "hq_stats_pack", "hq_stats_unpack", "hq_mma_peak_probe"]

# numpy view of hq_range_state (64 bytes)
RANGE_STATE_DTYPE = np.dtype([("acc_min", "<i4"), ("acc_max", "<i4"), ("acc_scale", "<f4"), ("step", "<u4"), ("q_min", "<f4"),
                              ("q_max", "<f4"), ("scale", "<f4"), ("inv_scale", "<f4"), ("zero_point", "<i4"), ("rounding", "<u4"), ("seed", "<u4"), ("dynamic_eta", "<f4"),
                              ("sat_below", "<u4"), ("sat_above", "<u4"), ("last_sat_below", "<u4"), ("last_sat_above", "<u4")])
assert RANGE_STATE_DTYPE.itemsize == 64
STATE_BYTES = RANGE_STATE_DTYPE.itemsize
INT32_MAX, INT32_MIN = 2**31 - 1, -2**31


class ConvDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("N", "H", "W", "C", "K", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w", "groups")]


class OpDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32), ("conv", C.POINTER(ConvDesc)),
                ("x", C.c_void_p), ("xq", C.c_void_p), ("w", C.c_void_p), ("bias", C.c_void_p), ("pw", C.c_void_p),
                ("w_scale", C.c_void_p)]


class HqError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


_lib = None


def lib():
    """Loads libhq.so; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2105_04246_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        L.hq_create.argtypes = [C.POINTER(vp), C.c_int]
        L.hq_destroy.argtypes = [vp]
        L.hq_status_string.argtypes = [C.c_int]; L.hq_status_string.restype = C.c_char_p
        L.hq_last_error.argtypes = [vp]; L.hq_last_error.restype = C.c_char_p
        L.hq_get_async_error.argtypes = [vp, vp, C.POINTER(i32)]
        L.hq_launch_count.argtypes = [vp]; L.hq_launch_count.restype = C.c_uint64
        L.hq_pair_launch_count.argtypes = [vp]; L.hq_pair_launch_count.restype = C.c_uint64
        L.hq_set_option.argtypes = [vp, C.c_char_p, i32]
        L.hq_weights_prepare.argtypes = [vp, vp, C.POINTER(ConvDesc), C.c_int, vp, C.POINTER(vp)]
        L.hq_weights_prepare_zp.argtypes = [vp, vp, C.POINTER(ConvDesc), C.c_int, vp, i32, C.POINTER(vp)]
        L.hq_linear_prepare.argtypes = [vp, vp, i32, i32, vp, i32, i32, C.POINTER(vp)]
        L.hq_linear_fwd_prepared.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
        L.hq_weights_release.argtypes = [vp, vp]
        L.hq_linear_fwd.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.hq_conv_fwd.argtypes = [vp, vp, C.POINTER(ConvDesc), vp, vp, vp, vp, vp, vp]
        L.hq_conv_bwd_data.argtypes = [vp, vp, C.POINTER(ConvDesc), vp, vp, vp, vp, vp, vp]
        L.hq_linear_wgrad.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
        L.hq_conv_wgrad.argtypes = [vp, vp, C.POINTER(ConvDesc), vp, vp, vp, vp, vp]
        L.hq_range_update.argtypes = [vp, vp, vp, i32, C.c_float]
        L.hq_dynamic_quant.argtypes = [vp, vp, C.POINTER(OpDesc), vp, vp, vp]
        L.hq_debug_accumulate.argtypes = [vp, vp, C.POINTER(OpDesc), vp, vp]
        L.hq_dynamic_quant_static.argtypes = [vp, vp, C.POINTER(OpDesc), vp, vp]
        L.hq_stats_pack.argtypes = [vp, vp, vp, i32, vp]
        L.hq_stats_unpack.argtypes = [vp, vp, vp, i32, vp]
        L.hq_mma_peak_probe.argtypes = [vp, vp, i32, i32, i32, C.POINTER(C.c_uint64)]
        for name in EXPORTS:
            if name not in ("hq_status_string", "hq_last_error", "hq_launch_count", "hq_pair_launch_count"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _ptr(x):
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return int(x)


def _stream(s):
    if s is None:
        return None
    if hasattr(s, "cuda_stream"):
        return s.cuda_stream
    return int(s)


def conv_desc(N, H, W, Cin, K, R=1, S=1, stride=1, pad=0, groups=1) -> ConvDesc:
    sh, sw = (stride, stride) if np.isscalar(stride) else stride
    ph, pw = (pad, pad) if np.isscalar(pad) else pad
    return ConvDesc(N, H, W, Cin, K, R, S, sh, sw, ph, pw, groups)


class PreparedWeights:
    def __init__(self, ctx: "Context", handle: int, desc: ConvDesc, direction: int):
        self.ctx, self.handle, self.desc, self.direction = ctx, handle, desc, direction

    def release(self):
        if self.handle:
            lib().hq_weights_release(self.ctx.handle, self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.release()
        except Exception:
            pass


class Context:
    """hq_ctx: one per device."""

    def __init__(self, device: int = 0):
        h = C.c_void_p()
        st = lib().hq_create(C.byref(h), int(device))
        if st != HQ_OK:
            raise HqError(st, lib().hq_status_string(st).decode())
        self.handle = h.value
        self.device = int(device)

    def close(self):
        if self.handle:
            lib().hq_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != HQ_OK:
            raise HqError(st, lib().hq_last_error(self.handle).decode())

    # ---- calls, named as in include/hq.h ------------------------------------------------------
    def weights_prepare(self, stream, desc: ConvDesc, direction: int, W, w_zero_point: int = 0) -> PreparedWeights:
        out = C.c_void_p()
        if w_zero_point:
            self._check(lib().hq_weights_prepare_zp(self.handle, _stream(stream), C.byref(desc), int(direction), _ptr(W), int(w_zero_point),
                                                    C.byref(out)))
        else:
            self._check(lib().hq_weights_prepare(self.handle, _stream(stream), C.byref(desc), int(direction), _ptr(W), C.byref(out)))
        return PreparedWeights(self, out.value, desc, int(direction))

    def linear_prepare(self, stream, N: int, K: int, W, w_zero_point: int = 0, max_M: int = 0) -> PreparedWeights:
        out = C.c_void_p()
        self._check(lib().hq_linear_prepare(self.handle, _stream(stream), int(N), int(K), _ptr(W), int(w_zero_point), int(max_M), C.byref(out)))
        return PreparedWeights(self, out.value, None, DIR_FWD)

    def linear_fwd_prepared(self, stream, M, X, xq, pw: PreparedWeights, w_scale, bias, Y, yq):
        self._check(lib().hq_linear_fwd_prepared(self.handle, _stream(stream), int(M), _ptr(X), _ptr(xq), pw.handle, _ptr(w_scale), _ptr(bias),
                                                 _ptr(Y), _ptr(yq)))

    def linear_fwd(self, stream, M, N, K, X, xq, W, w_scale, bias, Y, yq):
        self._check(lib().hq_linear_fwd(self.handle, _stream(stream), M, N, K, _ptr(X), _ptr(xq), _ptr(W), _ptr(w_scale), _ptr(bias),
                                        _ptr(Y), _ptr(yq)))

    def linear_wgrad(self, stream, M, N, K, dY, dyq, X, xq, GW):
        self._check(lib().hq_linear_wgrad(self.handle, _stream(stream), M, N, K, _ptr(dY), _ptr(dyq), _ptr(X), _ptr(xq), _ptr(GW)))

    def conv_wgrad(self, stream, desc, dY, dyq, X, xq, GW):
        self._check(lib().hq_conv_wgrad(self.handle, _stream(stream), C.byref(desc), _ptr(dY), _ptr(dyq), _ptr(X), _ptr(xq), _ptr(GW)))

    def conv_fwd(self, stream, desc, X, xq, pw: PreparedWeights, w_scale, Y, yq):
        self._check(lib().hq_conv_fwd(self.handle, _stream(stream), C.byref(desc), _ptr(X), _ptr(xq), pw.handle, _ptr(w_scale), _ptr(Y),
                                      _ptr(yq)))

    def conv_bwd_data(self, stream, desc, dY, dyq, pw: PreparedWeights, w_scale, dX, dxq):
        self._check(lib().hq_conv_bwd_data(self.handle, _stream(stream), C.byref(desc), _ptr(dY), _ptr(dyq), pw.handle, _ptr(w_scale),
                                           _ptr(dX), _ptr(dxq)))

    def range_update(self, stream, states, count: int, eta: float):
        self._check(lib().hq_range_update(self.handle, _stream(stream), _ptr(states), int(count), float(eta)))

    def dynamic_quant(self, stream, op: OpDesc, workspace, Y, yq):
        self._check(lib().hq_dynamic_quant(self.handle, _stream(stream), C.byref(op), _ptr(workspace), _ptr(Y), _ptr(yq)))

    def dynamic_quant_static(self, stream, op: OpDesc, Y, yq):
        """hq_dynamic_quant with the library's built-in workspace: for callers that cannot allocate
        device memory (see include/hq.h).  Shares one array per device; do not overlap calls."""
        self._check(lib().hq_dynamic_quant_static(self.handle, _stream(stream), C.byref(op), _ptr(Y), _ptr(yq)))

    def stats_pack(self, stream, states, count: int, buf):
        self._check(lib().hq_stats_pack(self.handle, _stream(stream), _ptr(states), int(count), _ptr(buf)))

    def stats_unpack(self, stream, states, count: int, buf):
        self._check(lib().hq_stats_unpack(self.handle, _stream(stream), _ptr(states), int(count), _ptr(buf)))

    def mma_peak_probe(self, stream, pair: int, bn: int, chunks: int) -> int:
        """Enqueues the MMA-only probe kernel; returns the 2 x MAC count of the launch."""
        ops = C.c_uint64(0)
        self._check(lib().hq_mma_peak_probe(self.handle, _stream(stream), int(pair), int(bn), int(chunks), C.byref(ops)))
        return int(ops.value)

    def debug_accumulate(self, stream, op: OpDesc, acc, yq):
        self._check(lib().hq_debug_accumulate(self.handle, _stream(stream), C.byref(op), _ptr(acc), _ptr(yq)))

    def get_async_error(self, stream=None) -> int:
        code = C.c_int32(0)
        st = lib().hq_get_async_error(self.handle, _stream(stream), C.byref(code))
        if st not in (HQ_OK, 6):
            self._check(st)
        return code.value

    def set_option(self, key: str, value: int):
        self._check(lib().hq_set_option(self.handle, key.encode(), int(value)))

    def launch_count(self) -> int:
        return int(lib().hq_launch_count(self.handle))

    def pair_launch_count(self) -> int:
        return int(lib().hq_pair_launch_count(self.handle))


def linear_op(M, N, K, X, xq, W, w_scale, bias=None, pw: PreparedWeights | None = None) -> OpDesc:
    """pw: weights from linear_prepare (N, K and W are then taken from the handle)."""
    op = OpDesc(OP_LINEAR, M, N, K, None, _ptr(X), _ptr(xq), _ptr(W), _ptr(bias), None if pw is None else pw.handle, _ptr(w_scale))
    op._keep = (pw,)
    return op


def conv_op(kind: int, desc: ConvDesc, X, xq, pw: PreparedWeights, w_scale) -> OpDesc:
    op = OpDesc(kind, 0, 0, 0, C.pointer(desc), _ptr(X), _ptr(xq), None, None, pw.handle, _ptr(w_scale))
    op._keep = (desc, pw)
    return op


# ---- range-state helpers (host-side packing of the plain-data struct) -------------------------------
ROUND_NEAREST_EVEN, ROUND_STOCHASTIC = 0, 1
COUNT_SATURATION = 0x100      # flag in `rounding`: count the outputs outside the grid (sat_below / sat_above)


def new_states(count: int, sr_seed: int | None = None) -> np.ndarray:
    """`count` empty states: no range yet (step 0), empty statistics slot.  sr_seed: None = round to nearest even,
    an integer = stochastic rounding with that seed for the tensors these states describe."""
    s = np.zeros(count, RANGE_STATE_DTYPE)
    s["acc_min"] = INT32_MAX
    s["acc_max"] = INT32_MIN
    if sr_seed is not None:
        s["rounding"] = ROUND_STOCHASTIC
        s["seed"] = int(sr_seed) & 0xFFFFFFFF
    return s


def input_state(scale: float, zero_point: int) -> np.ndarray:
    """State describing a layer INPUT: only scale and zero_point are read."""
    s = new_states(1)
    s["scale"] = np.float32(scale)
    s["zero_point"] = int(zero_point)
    return s


def states_to_device(states: np.ndarray, device="cuda"):
    import torch
    return torch.from_numpy(states.view(np.uint8).reshape(-1).copy()).to(device)


def states_from_device(t) -> np.ndarray:
    return t.detach().cpu().numpy().view(RANGE_STATE_DTYPE).copy()
