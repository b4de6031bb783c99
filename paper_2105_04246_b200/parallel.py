"""Data parallelism over the batch: the one exchange step the method needs.

Each rank runs the layer kernels on its shard of the batch with the same (replicated) range state.
The only quantity that couples the shards is the per-tensor statistic of Sec. 4.1 of the paper --
min and max of the unquantized output over the WHOLE tensor -- so before the range update every rank
needs the extremes over all shards.  Integer min/max is order independent, hence after this exchange
every rank applies Eq. 2-3 to identical numbers and the replicated states stay bit-identical.

Plumbing only (torch.distributed over NCCL on GPUs, gloo on CPU); no arithmetic of the method.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

STATE_WORDS = 12          # hq_range_state is 12 x 32-bit words; words 0 and 1 are acc_min and acc_max


def allreduce_stats(states: torch.Tensor, group=None) -> None:
    """In place: acc_min <- min over ranks, acc_max <- max over ranks, for every state.

    `states` is the byte (uint8) or int32 tensor holding an array of hq_range_state.  One collective:
    the maxima travel as their bitwise complement (an order-reversing map without overflow), so a single
    MIN all-reduce serves both columns.  An empty slot {INT32_MAX, INT32_MIN} is the identity.
    """
    words = states.view(torch.int32).view(-1, STATE_WORDS)
    buf = torch.stack([words[:, 0], torch.bitwise_not(words[:, 1])]).contiguous()
    dist.all_reduce(buf, op=dist.ReduceOp.MIN, group=group)
    words[:, 0] = buf[0]
    words[:, 1] = torch.bitwise_not(buf[1])
