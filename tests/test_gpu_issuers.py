"""Several MMA-issuing warps per CTA: the accumulator hand-off between issuers and epilogue groups must give the same
bytes as one issuer and must never stall.  The shape is a 1x1 layer with a long reduction and few output channels, many
tiles per CTA (the layer kernel then runs three issuers over eight narrow accumulator buffers and an operand ring as deep
as those buffers), repeated many times on both paths; the real-valued first pass of the dynamic path is the slowest
epilogue and lets the issuers run furthest ahead."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2105_04246_b200 import hq, synth
from tests.harness import oracle_range_from_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = hq.Context(0)
    yield c
    c.close()


def test_three_issuers_match_one_issuer_and_never_stall(ctx):
    dev = torch.device("cuda", ctx.device)
    N, H, W, C, K = 64, 56, 56, 144, 24          # 200704 output pixels: 1568 row tiles on 148 CTAs
    r = synth.rng(515)
    x = synth.relu_activations(r, (N, H, W, C))
    w = synth.weights(r, (K, 1, 1, C))
    d = hq.conv_desc(N, H, W, C, K, 1, 1, 1, 0, 1)
    xd = torch.from_numpy(x.q).to(dev)
    Wd = torch.from_numpy(w.q).to(dev)
    wsc = torch.tensor([w.scale], dtype=torch.float32, device=dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    outs = {}
    for issuers in (1, 3):
        ctx.set_option("issuers", issuers)
        try:
            pw = ctx.weights_prepare(None, d, hq.DIR_FWD, Wd)
            yq = hq.states_to_device(hq.new_states(1), dev)
            y = torch.empty((N, H, W, K), dtype=torch.int8, device=dev)
            ws = torch.empty((N, H, W, K), dtype=torch.float32, device=dev)
            op = hq.conv_op(hq.OP_CONV_FWD, d, xd, xq, pw, wsc)
            ctx.dynamic_quant(None, op, ws, y, yq)          # iteration 0: sets the range
            ctx.range_update(None, yq, 1, 0.9)
            first = None
            for it in range(120):
                ctx.dynamic_quant(None, op, ws, y, yq)
                ctx.conv_fwd(None, d, xd, xq, pw, wsc, y, yq)
                if it % 40 == 0:
                    torch.cuda.synchronize(dev)
                    assert ctx.get_async_error() == 0, f"device wait expired with {issuers} issuer(s), iteration {it}"
                    cur = y.cpu().numpy().copy()
                    if first is None:
                        first = cur
                    assert np.array_equal(cur, first), "the same inputs and range gave different codes"
            torch.cuda.synchronize(dev)
            assert ctx.get_async_error() == 0
            outs[issuers] = (first, hq.states_from_device(yq)[0].copy())
        finally:
            ctx.set_option("issuers", 3)
    assert np.array_equal(outs[1][0], outs[3][0])
    # and the oracle on a sample of pixels: accumulate, then quantize with the state the kernel used
    st = outs[3][1]
    rows = np.unique(np.concatenate([np.arange(0, 300), r.integers(0, N * H * W, 2000), np.arange(N * H * W - 300, N * H * W)]))
    xs = x.q.reshape(-1, C)[rows].astype(np.int64) - x.zero_point
    acc = xs @ w.q.reshape(K, C).astype(np.int64).T
    s_acc = O.acc_scale(x.scale, w.scale)
    want = O.quantize(np.ascontiguousarray(acc.astype(np.int32)), s_acc, oracle_range_from_gpu(st))
    assert np.array_equal(outs[3][0].reshape(-1, K)[rows], want)
