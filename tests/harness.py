"""Test-side drivers: one layer run on the GPU through the C-ABI binding, and the same layer on
the CPU oracle.  Only tests (and the smoke check) use this module."""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
from paper_2105_04246_b200 import hq
from paper_2105_04246_b200.synth import QTensor


GUARD_BYTES = 4096            # sentinel band on both sides of every output the kernels write
GUARD_BYTE = 0xA5


class Guarded:
    """An output tensor carved out of a larger byte buffer with GUARD_BYTES of a sentinel value before and after it.
    check() fails if a kernel wrote outside the tensor (the memory checker of the toolkit is not available on the
    machines these tests run on, so stores past the end of ragged tiles would otherwise go unseen)."""

    def __init__(self, shape, dtype, dev, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = n
        self.buf = torch.full((2 * GUARD_BYTES + ((n + 15) // 16) * 16,), GUARD_BYTE, dtype=torch.uint8, device=dev)
        self.t = self.buf[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)     # 16-byte aligned like a fresh allocation
        assert self.t.data_ptr() % 16 == 0
        if fill is not None:
            self.t.fill_(fill)

    def check(self):
        lo = self.buf[:GUARD_BYTES]
        hi = self.buf[GUARD_BYTES + self.nbytes:]
        assert bool((lo == GUARD_BYTE).all()), "a kernel wrote BEFORE the start of its output tensor"
        assert bool((hi == GUARD_BYTE).all()), "a kernel wrote PAST the end of its output tensor"
        return self.t


class GpuLayer:
    """kind: 'linear' | 'conv_fwd' | 'conv_bwd'.  For conv kinds `shape` is a dict of conv_desc arguments."""

    def __init__(self, ctx: hq.Context, kind: str, W: QTensor, shape: dict | None = None, bias: np.ndarray | None = None, eta: float = 0.9,
                 sr_seed: int | None = None, count_sat: bool = False, prepared: bool = False, max_M: int = 0):
        """W.zero_point != 0: asymmetric weights (prepared with their zero point).  count_sat: the output state asks for the
        saturation counts.  prepared (linear): weights go through hq_linear_prepare / hq_linear_fwd_prepared."""
        self.ctx, self.kind, self.eta = ctx, kind, eta
        self.dev = torch.device("cuda", ctx.device)
        self.W = torch.from_numpy(np.ascontiguousarray(W.q)).to(self.dev)
        self.w_scale = torch.tensor([W.scale], dtype=torch.float32, device=self.dev)
        self.bias = None if bias is None else torch.from_numpy(np.ascontiguousarray(bias, dtype=np.int32)).to(self.dev)
        st = hq.new_states(1, sr_seed)                                        # sr_seed: stochastic rounding of this layer's output
        if count_sat:
            st["rounding"] |= hq.COUNT_SATURATION
        self.yq = hq.states_to_device(st, self.dev)
        self.stream = torch.cuda.current_stream(self.dev)
        if kind == "linear":
            self.N, self.K = W.q.shape
            self.pw = None
            if prepared or W.zero_point != 0:
                self.pw = ctx.linear_prepare(self.stream, self.N, self.K, self.W, W.zero_point, max_M)
        else:
            self.desc = hq.conv_desc(**shape)
            self.pw = ctx.weights_prepare(self.stream, self.desc, hq.DIR_FWD if kind == "conv_fwd" else hq.DIR_BWD_DATA, self.W, W.zero_point)
            d = self.desc
            Ho = (d.H + 2 * d.pad_h - d.R) // d.stride_h + 1
            Wo = (d.W + 2 * d.pad_w - d.S) // d.stride_w + 1
            self.in_shape = (d.N, d.H, d.W, d.C) if kind == "conv_fwd" else (d.N, Ho, Wo, d.K)
            self.out_shape = (d.N, Ho, Wo, d.K) if kind == "conv_fwd" else (d.N, d.H, d.W, d.C)

    def _put(self, x: QTensor):
        xd = torch.from_numpy(np.ascontiguousarray(x.q)).to(self.dev)
        xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), self.dev)
        if self.kind == "linear":
            assert x.q.shape[1] == self.K
            out_shape = (x.q.shape[0], self.N)
        else:
            assert tuple(x.q.shape) == self.in_shape, (x.q.shape, self.in_shape)
            out_shape = self.out_shape
        return xd, xq, out_shape

    def _op(self, xd, xq):
        if self.kind == "linear":
            return hq.linear_op(xd.shape[0], self.N, self.K, xd, xq, self.W, self.w_scale, self.bias, pw=self.pw)
        return hq.conv_op(hq.OP_CONV_FWD if self.kind == "conv_fwd" else hq.OP_CONV_BWD_DATA, self.desc, xd, xq, self.pw, self.w_scale)

    def state(self) -> np.ndarray:
        return hq.states_from_device(self.yq)[0]

    def set_state(self, st: np.ndarray):
        arr = np.array([st], dtype=hq.RANGE_STATE_DTYPE)
        self.yq.copy_(torch.from_numpy(arr.view(np.uint8).reshape(-1).copy()))

    def accumulate(self, x: QTensor):
        """Debug hook: int32 accumulator and its min/max (does not disturb the layer's own state)."""
        xd, xq, out_shape = self._put(x)
        g_acc = Guarded(out_shape, torch.int32, self.dev)
        acc = g_acc.t
        tmp = hq.states_to_device(hq.new_states(1), self.dev)
        self.ctx.debug_accumulate(self.stream, self._op(xd, xq), acc, tmp)
        torch.cuda.synchronize(self.dev)
        g_acc.check()
        st = hq.states_from_device(tmp)[0]
        return acc.cpu().numpy(), int(st["acc_min"]), int(st["acc_max"]), float(st["acc_scale"])

    def dynamic(self, x: QTensor):
        xd, xq, out_shape = self._put(x)
        g_ws, g_y = Guarded(out_shape, torch.float32, self.dev), Guarded(out_shape, torch.int8, self.dev, fill=99)
        ws, y = g_ws.t, g_y.t
        self.ctx.dynamic_quant(self.stream, self._op(xd, xq), ws, y, self.yq)
        torch.cuda.synchronize(self.dev)
        g_ws.check()
        g_y.check()
        return y.cpu().numpy(), ws.cpu().numpy()

    def hindsight(self, x: QTensor, update: bool = True):
        xd, xq, out_shape = self._put(x)
        g_y = Guarded(out_shape, torch.int8, self.dev, fill=99)
        y = g_y.t
        if self.kind == "linear" and self.pw is not None:
            self.ctx.linear_fwd_prepared(self.stream, xd.shape[0], xd, xq, self.pw, self.w_scale, self.bias, y, self.yq)
        elif self.kind == "linear":
            self.ctx.linear_fwd(self.stream, xd.shape[0], self.N, self.K, xd, xq, self.W, self.w_scale, self.bias, y, self.yq)
        elif self.kind == "conv_fwd":
            self.ctx.conv_fwd(self.stream, self.desc, xd, xq, self.pw, self.w_scale, y, self.yq)
        else:
            self.ctx.conv_bwd_data(self.stream, self.desc, xd, xq, self.pw, self.w_scale, y, self.yq)
        torch.cuda.synchronize(self.dev)
        g_y.check()
        stats = self.state()
        if update:
            self.ctx.range_update(self.stream, self.yq, 1, self.eta)
            torch.cuda.synchronize(self.dev)
        return y.cpu().numpy(), (int(stats["acc_min"]), int(stats["acc_max"]), float(stats["acc_scale"]))

    def step(self, x: QTensor):
        """Iteration 0: dynamic path; afterwards: in-hindsight layer call + range update."""
        if int(self.state()["step"]) == 0:
            return self.dynamic(x)[0]
        return self.hindsight(x)[0]


class OracleLayer:
    def __init__(self, kind: str, W: QTensor, shape: dict | None = None, bias: np.ndarray | None = None, eta: float = 0.9,
                 sr_seed: int | None = None):
        self.kind, self.W, self.bias = kind, W, bias
        self.layer = O.Layer(eta, sr_seed)
        self.desc = None if kind == "linear" else O.conv_desc(shape["N"], shape["H"], shape["W"], shape["Cin"], shape["K"], shape.get("R", 1),
                                                              shape.get("S", 1), shape.get("stride", 1), shape.get("pad", 0),
                                                              shape.get("groups", 1))

    def accumulate(self, x: QTensor) -> np.ndarray:
        if self.kind == "linear":
            return O.linear_acc(x.q, x.zero_point, self.W.q, self.W.zero_point, self.bias)
        if self.kind == "conv_fwd":
            return O.conv_fwd_acc(self.desc, x.q, x.zero_point, self.W.q, self.W.zero_point)
        return O.conv_bwd_data_acc(self.desc, x.q, x.zero_point, self.W.q, self.W.zero_point)

    def s_acc(self, x: QTensor) -> float:
        return O.acc_scale(x.scale, self.W.scale)

    def step(self, x: QTensor, force_state: O.Range | None = None) -> O.StepResult:
        return self.layer.step(self.accumulate(x), self.s_acc(x), force_state)


def oracle_range_from_gpu(st: np.ndarray) -> O.Range:
    return O.Range(float(st["q_min"]), float(st["q_max"]), float(st["scale"]), float(st["inv_scale"]), int(st["zero_point"]), int(st["step"]))


def assert_state_close(gpu_st: np.ndarray, orc: O.Range, rel: float = 1e-6):
    for name in ("q_min", "q_max", "scale", "inv_scale"):
        a, b = float(gpu_st[name]), float(getattr(orc, name))
        assert abs(a - b) <= rel * max(abs(a), abs(b), 1e-30), (name, a, b)
    assert int(gpu_st["zero_point"]) == orc.zero_point, (int(gpu_st["zero_point"]), orc.zero_point)
    assert int(gpu_st["step"]) == orc.step
