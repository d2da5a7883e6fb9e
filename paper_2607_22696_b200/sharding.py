"""Head sharding of one 3D-DSA problem over several GPUs.

Every head has its own q/k/v channels and its own offsets, and no sample of one head reads
another head, so a problem splits over heads with no exchange inside the operator: rank r of
G takes heads [r*h/G, (r+1)*h/G) of all tokens and calls the single-GPU entry points on its
slice; outputs and gradients of the full problem are the concatenation of the ranks' results
along the head axis.  If the surrounding model is sharded over tokens instead, the
conversion is one all-to-all before and after the operator, outside this library.

This module holds only the index arithmetic and the slicing / reassembly of tensors in the
library's layouts; it launches nothing.
"""
from __future__ import annotations

from typing import Sequence, Tuple

import torch


def head_range(heads: int, world: int, rank: int) -> Tuple[int, int]:
    """Heads [lo, hi) of rank `rank` of `world`; the first heads % world ranks take one more."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    base, extra = divmod(heads, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_heads(t: torch.Tensor, world: int, rank: int, head_axis: int = 3) -> torch.Tensor:
    """The contiguous slice of `t` ([T,H,W,heads,...]: rows, offsets, lse) that rank `rank` owns."""
    lo, hi = head_range(t.shape[head_axis], world, rank)
    return t.narrow(head_axis, lo, hi - lo).contiguous()


def unshard_heads(parts: Sequence[torch.Tensor], head_axis: int = 3) -> torch.Tensor:
    """Inverse of shard_heads over all ranks, in rank order."""
    return torch.cat(list(parts), dim=head_axis)
