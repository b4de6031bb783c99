"""The statistics exchange of batch-sharded data parallelism on one GPU: the library's pack / unpack kernels against
the same packing done with tensor operations, and a one-rank NCCL group through a captured step."""
import numpy as np
import pytest
import torch

from paper_2105_04246_b200 import hq

pytestmark = pytest.mark.gpu


def test_pack_and_unpack_kernels():
    dev = torch.device("cuda", 0)
    ctx = hq.Context(0)
    r = np.random.default_rng(5)
    n = 41
    st = hq.new_states(n)
    st["acc_min"] = r.integers(-2**31, 2**31, size=n)
    st["acc_max"] = r.integers(-2**31, 2**31, size=n)
    st["acc_min"][3], st["acc_max"][3] = hq.INT32_MAX, hq.INT32_MIN          # an empty slot
    st["q_min"] = r.normal(size=n)
    d = hq.states_to_device(st, dev)
    buf = torch.full((2 * n + 8,), 12345, dtype=torch.int32, device=dev)
    ctx.stats_pack(None, d, n, buf)
    torch.cuda.synchronize()
    b = buf.cpu().numpy()
    assert np.array_equal(b[:n], st["acc_min"]) and np.array_equal(b[n:2 * n], ~st["acc_max"]) and (b[2 * n:] == 12345).all()
    assert (int(b[3]), int(b[n + 3])) == (hq.INT32_MAX, hq.INT32_MAX)          # identity of the MIN reduction in both columns
    # another rank's pair merged in by hand, then unpacked
    other_min, other_max = st["acc_min"] // 2, st["acc_max"] // 2
    merged = np.concatenate([np.minimum(b[:n], other_min), np.minimum(b[n:2 * n], ~other_max)]).astype(np.int32)
    ctx.stats_unpack(None, d, n, torch.from_numpy(merged).to(dev))
    torch.cuda.synchronize()
    got = hq.states_from_device(d)
    assert np.array_equal(got["acc_min"], np.minimum(st["acc_min"], other_min))
    assert np.array_equal(got["acc_max"], np.maximum(st["acc_max"], other_max))
    for f in ("q_min", "step", "scale", "zero_point", "seed"):
        assert np.array_equal(got[f], st[f])                                    # nothing else touched
    assert ctx.get_async_error() == 0
    ctx.close()
