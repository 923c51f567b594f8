"""Sequence-sharded forward pass: every rank holds a slice of the positions.

K' = E K and V' = F V (arxiv 2306.15799, Eq. (2)) are sums over positions, so a rank computes its part
from its slice of K, V and the matching columns of E, F; one all-reduce (sum) of the fp32 block
[2][B*H][k][d] over the ranks (NCCL through torch.distributed) completes them, and the feature maps, the
associative product and the division are local to a rank's queries.  Only orchestration lives here:
every arithmetic step runs inside the CUDA library.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding


def shard_bounds(N: int, world: int, rank: int, multiple: int = 8):
    """[begin, end) of rank's contiguous slice of N positions; every slice but the last is a multiple of
    `multiple` positions long (the tensor-core kernels want slices that are multiples of 8)."""
    if not 0 <= rank < world:
        raise ValueError("rank %d outside a world of %d" % (rank, world))
    units = (N + multiple - 1) // multiple
    b = (units * rank // world) * multiple
    e = (units * (rank + 1) // world) * multiple
    return min(b, N), min(e, N)


def forward_sequence_sharded(Q, K, V, E, F, W, variant, group=None, out=None, stream=None, layout="bhnd"):
    """One rank's share of a forward pass sharded over the sequence.

    Q, K, V: this rank's positions ([B,H,n,d], or [B,n,H,d] with layout='bnhd'); E, F: the matching
    columns, dense [k,n]; W: [m,d] or None.  Returns this rank's rows of the output.  Without an initialised
    process group (or with a group of one) the sum over ranks is skipped.
    """
    m = W.shape[0] if W is not None else 0
    binding.flurka_forward_partial(K, V, E, F, variant, m=m, stream=stream, layout=layout)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        block = binding.flurka_partial_sums()
        if stream is not None:
            with torch.cuda.stream(stream):
                dist.all_reduce(block, op=dist.ReduceOp.SUM, group=group)
        else:
            dist.all_reduce(block, op=dist.ReduceOp.SUM, group=group)
    return binding.flurka_forward_finish(Q, W, variant, E.shape[-2], out=out, stream=stream, layout=layout)
