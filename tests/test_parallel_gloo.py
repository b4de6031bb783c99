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


def _train_worker(rank, world, port, accs, s_acc, eta, out):
    """Each rank sees its half of every iteration's accumulator tensor; statistics are merged, then Eq. 2-3 is applied locally."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q = O.Range()
    st = hq.new_states(1)
    for acc in accs:
        shard = np.array_split(acc, world, axis=0)[rank]
        st["acc_min"][0], st["acc_max"][0] = O.minmax(shard)
        t = torch.from_numpy(st.view(np.uint8).reshape(-1).copy())
        parallel.allreduce_stats(t)
        merged = t.numpy().view(hq.RANGE_STATE_DTYPE)
        O.range_update(q, int(merged["acc_min"][0]), int(merged["acc_max"][0]), s_acc, eta)
        st["acc_min"][0], st["acc_max"][0] = hq.INT32_MAX, hq.INT32_MIN       # the update empties the slot
    out[rank] = q.astuple()
    dist.destroy_process_group()


def test_replicated_range_state_stays_identical_over_iterations():
    """Five iterations on two ranks: after every exchange both ranks apply the moving average of Eq. 2-3 to the same
    pair, so their range states stay bit-identical and equal the state of one process that saw the whole batch."""
    r = synth.rng(301)
    accs = [(r.integers(-10**5, 10**5, size=(16, 40)) * (1.0 + 0.3 * t)).astype(np.int32) for t in range(5)]
    s_acc, eta = 3.0e-4, 0.9
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_train_worker, args=(2, _free_port(), accs, s_acc, eta, out), nprocs=2, join=True)
    whole = O.Range()
    for acc in accs:
        O.range_update(whole, *O.minmax(acc), s_acc, eta)
    assert out[0] == out[1] == whole.astuple()
    assert whole.step == 5
