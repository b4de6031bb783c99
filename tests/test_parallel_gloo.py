"""World-size-2 check (gloo, CPU) of the statistics exchange used for batch sharding."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as O
from paper_2105_04246_b200 import hq, parallel, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    st = hq.new_states(3)
    # state 0: both ranks saw data; state 1: only rank 1 did; state 2: nobody did
    st["acc_min"][0], st["acc_max"][0] = (-50 - rank * 100, 70 + rank * 5)
    if rank == 1:
        st["acc_min"][1], st["acc_max"][1] = (-2**31, 2**31 - 1)
    t = torch.from_numpy(st.view(np.uint8).reshape(-1).copy())
    parallel.allreduce_stats(t)
    out[rank] = t.numpy().copy()
    dist.destroy_process_group()


def test_stats_exchange_world_size_2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    a = out[0].view(hq.RANGE_STATE_DTYPE)
    b = out[1].view(hq.RANGE_STATE_DTYPE)
    assert a.tobytes() == b.tobytes()                     # replicated state stays identical
    assert (int(a["acc_min"][0]), int(a["acc_max"][0])) == (-150, 75)
    assert (int(a["acc_min"][1]), int(a["acc_max"][1])) == (-2**31, 2**31 - 1)
    assert (int(a["acc_min"][2]), int(a["acc_max"][2])) == (hq.INT32_MAX, hq.INT32_MIN)   # still empty
    assert float(a["q_min"][0]) == 0.0 and int(a["step"][0]) == 0                         # nothing else touched


def test_sharded_statistics_equal_whole_tensor_statistics():
    """The oracle's min/max over a whole batch equals the merge of the per-shard extremes."""
    r = synth.rng(300)
    acc = r.integers(-10**6, 10**6, size=(8, 50)).astype(np.int32)
    shards = [O.minmax(acc[:4]), O.minmax(acc[4:])]
    assert (min(s[0] for s in shards), max(s[1] for s in shards)) == O.minmax(acc)
