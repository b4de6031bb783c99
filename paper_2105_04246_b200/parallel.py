"""Batch-sharded data parallelism for the in-hindsight layer path.

Each rank runs the layer calls on its slice of the batch with the full int8 weights and the same
(replicated) range states.  Sec. 4.1 takes min/max over the WHOLE tensor, so the one exchange of the
method is the statistics: before hq_range_update the per-rank slots {acc_min, acc_max} of all states are
merged with ONE int32 MIN all-reduce (the maxima travel as their bitwise complement), after which every
rank applies Eq. 2-3 to identical numbers and the replicated states stay bit-identical.

On CUDA the pack / unpack steps are the library's own kernels (hq_stats_pack / hq_stats_unpack) enqueued on
the caller's stream around the NCCL collective, so a whole step -- layers, exchange, update -- can be
captured into one CUDA graph.  On CPU tensors (the gloo test) the same packing is done with tensor ops.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

STATE_WORDS = 16          # hq_range_state is 16 x 32-bit words; words 0 and 1 are acc_min and acc_max


def allreduce_stats(states: torch.Tensor, group=None) -> None:
    """In place, host-side packing (CPU tensors): acc_min <- min over ranks, acc_max <- max over ranks."""
    words = states.view(torch.int32).view(-1, STATE_WORDS)
    buf = torch.stack([words[:, 0], torch.bitwise_not(words[:, 1])]).contiguous()
    dist.all_reduce(buf, op=dist.ReduceOp.MIN, group=group)
    words[:, 0] = buf[0]
    words[:, 1] = torch.bitwise_not(buf[1])


class StatsExchange:
    """The exchange step on CUDA: pack kernel, one NCCL MIN all-reduce of 2 * count int32, unpack kernel, all on the
    stream that is current when exchange() is called (inside a CUDA-graph capture they become graph nodes)."""

    def __init__(self, ctx, count: int, device, group=None):
        self.ctx, self.count, self.group = ctx, int(count), group
        self.buf = torch.empty(2 * self.count, dtype=torch.int32, device=device)

    def __call__(self, stream, states: torch.Tensor) -> None:
        self.ctx.stats_pack(stream, states, self.count, self.buf)
        dist.all_reduce(self.buf, op=dist.ReduceOp.MIN, group=self.group)      # runs on torch's current stream == `stream`
        self.ctx.stats_unpack(stream, states, self.count, self.buf)
