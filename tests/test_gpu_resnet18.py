"""The ResNet-18-shaped stack (every convolution at 224x224 input plus the classifier, forward and
backward data) at a reduced batch: every output element of all 41 layer calls against the oracle over
three iterations (dynamic initialisation, then two in-hindsight iterations with range updates)."""
import numpy as np
import pytest

import bench
from paper_2105_04246_b200 import hq, synth
from tests.harness import GpuLayer, OracleLayer, assert_state_close

pytestmark = pytest.mark.gpu


def test_resnet18_stack_batch4_three_iterations():
    ctx = hq.Context(0)
    layers, _ = bench.workload_layers("cfg5", 32)          # batch 128 / 32 = 4
    r = synth.rng(500)
    for kind, s, recipe in layers:
        xsh, ysh, wsh = bench.layer_shapes(kind, s)
        if kind == "linear":
            W, shape = synth.uniform_int8(r, wsh, scale=0.01), None
        else:
            W = synth.weights(r, wsh)
            shape = dict(N=s.N, H=s.H, W=s.W, Cin=s.C, K=s.K, R=s.R, S=s.S, stride=s.stride, pad=s.pad, groups=s.groups)
        g, o = GpuLayer(ctx, kind, W, shape), OracleLayer(kind, W, shape)
        for t in range(3):
            x = bench.make_input(recipe, r, xsh)
            x.scale *= float(np.exp(r.normal(0.0, 0.3)))    # range drift between iterations
            y, res = g.step(x), o.step(x)
            assert y.shape == tuple(ysh)
            bad = int((y != res.q).sum())
            assert bad == 0, f"{s.name} iteration {t}: {bad} of {y.size} int8 codes differ"
            assert_state_close(g.state(), o.layer.state)
        del g
    assert ctx.get_async_error() == 0
    ctx.close()
