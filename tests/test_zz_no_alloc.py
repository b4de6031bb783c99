"""hq_dynamic_quant_static: the dynamic path for callers that cannot allocate device memory
(allocator callbacks, loops that must stay out of the allocator, processes with a fixed memory
budget).  Its
workspace is a fixed array inside the library, so its results must equal hq_dynamic_quant's,
also when the shared array still holds the previous call's values.

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2105_04246_b200 import hq, synth
from tests.harness import Guarded

pytestmark = pytest.mark.gpu


def _run(ctx, dev, op_maker, out_shape, static):
    g_y = Guarded(out_shape, torch.int8, dev, fill=77)      # sentinel bands around the output: nothing may be written outside it
    y = g_y.t
    yq = hq.states_to_device(hq.new_states(1), dev)
    op = op_maker()
    if static:
        ctx.dynamic_quant_static(None, op, y, yq)
    else:
        ws = torch.empty(out_shape, dtype=torch.float32, device=dev)
        ctx.dynamic_quant(None, op, ws, y, yq)
    torch.cuda.synchronize(dev)
    g_y.check()
    return y.cpu().numpy(), hq.states_from_device(yq)[0]


def test_static_workspace_matches_caller_workspace_twice_in_a_row():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = hq.Context(0)
    r = synth.rng(900)
    # call 1: a 3x3 convolution; call 2: a smaller linear layer, so stale values stay behind it in the array
    shape = dict(N=2, H=12, W=12, Cin=64, K=64, R=3, S=3, stride=1, pad=1)
    desc = hq.conv_desc(**shape)
    Wc = synth.weights(r, (64, 3, 3, 64))
    xc = synth.relu_activations(r, (2, 12, 12, 64))
    Wc_d = torch.from_numpy(Wc.q).to(dev); xc_d = torch.from_numpy(xc.q).to(dev)
    wsc = torch.tensor([Wc.scale], dtype=torch.float32, device=dev)
    xcq = hq.states_to_device(hq.input_state(xc.scale, xc.zero_point), dev)
    pw = ctx.weights_prepare(None, desc, hq.DIR_FWD, Wc_d)
    Wl = synth.uniform_int8(r, (40, 64), scale=0.01)
    xl = synth.uniform_int8(r, (100, 64), scale=0.05, zero_point=3)
    Wl_d = torch.from_numpy(Wl.q).to(dev); xl_d = torch.from_numpy(xl.q).to(dev)
    wsl = torch.tensor([Wl.scale], dtype=torch.float32, device=dev)
    xlq = hq.states_to_device(hq.input_state(xl.scale, xl.zero_point), dev)

    conv_op = lambda: hq.conv_op(hq.OP_CONV_FWD, desc, xc_d, xcq, pw, wsc)
    lin_op = lambda: hq.linear_op(100, 40, 64, xl_d, xlq, Wl_d, wsl)
    n0 = ctx.launch_count()
    for op_maker, out_shape in ((conv_op, (2, 12, 12, 64)), (lin_op, (100, 40)), (conv_op, (2, 12, 12, 64))):
        y_ref, st_ref = _run(ctx, dev, op_maker, out_shape, static=False)
        y_sta, st_sta = _run(ctx, dev, op_maker, out_shape, static=True)
        assert np.array_equal(y_sta, y_ref)                       # bit-exact, as in the other parity tests
        assert st_sta.tobytes() == st_ref.tobytes()
        assert (y_sta != 77).any()
    assert ctx.launch_count() > n0
    # larger than the built-in workspace: refused before any launch
    n1 = ctx.launch_count()
    with pytest.raises(hq.HqError) as e:
        ctx.dynamic_quant_static(None, hq.linear_op(8192, 1024, 64, xl_d, xlq, Wl_d, wsl), xl_d, xlq)
    assert e.value.status == 2 and "workspace" in str(e.value)
    assert ctx.launch_count() == n1
    # scratch the context does not hold is not grown by this call: refused, nothing launched
    big_w = torch.zeros((5000, 64), dtype=torch.int8, device=dev)
    with pytest.raises(hq.HqError) as e:
        ctx.dynamic_quant_static(None, hq.linear_op(64, 5000, 64, xl_d, xlq, big_w, wsl), xl_d, xlq)
    assert e.value.status == 2 and "may not allocate" in str(e.value)
    odd_w = torch.zeros((40, 24), dtype=torch.int8, device=dev)
    with pytest.raises(hq.HqError) as e:
        ctx.dynamic_quant_static(None, hq.linear_op(100, 40, 24, xl_d, xlq, odd_w, wsl), xl_d, xlq)
    assert e.value.status == 2 and "may not allocate" in str(e.value)
    assert ctx.launch_count() == n1
    assert ctx.get_async_error() == 0
    pw.release()
    ctx.close()
