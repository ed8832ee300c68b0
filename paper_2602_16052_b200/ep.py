"""Expert-parallel plumbing around the layer: which experts a rank holds, and the reduction of the ranks'
partial outputs.  No method arithmetic lives here: every rank runs the same routing on the same hidden states
(the router is replicated), streams only its resident kept experts and returns a partial sum; the layer output
is the sum of the partial sums (one exchange step per layer, [M, d] fp32).
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def expert_range(rank: int, world: int, n_experts: int) -> Tuple[int, int]:
    """(first, count) of the contiguous block of experts that `rank` of `world` holds.  The blocks cover
    0..n_experts-1 exactly once; the first n_experts % world ranks hold one expert more."""
    if not (0 <= rank < world) or world > n_experts:
        raise ValueError("need 0 <= rank < world <= n_experts")
    base, extra = divmod(n_experts, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def owner_of(expert: int, world: int, n_experts: int) -> int:
    """Rank that holds `expert` under expert_range."""
    for r in range(world):
        first, count = expert_range(r, world, n_experts)
        if first <= expert < first + count:
            return r
    raise ValueError("expert out of range")


def sum_in_rank_order(partials: List[torch.Tensor]) -> torch.Tensor:
    """partials[0] + partials[1] + ... added one after the other in fp32: a fixed order, so the result does
    not depend on how a collective happens to combine them."""
    acc = partials[0].to(torch.float32).clone()
    for p in partials[1:]:
        acc += p.to(torch.float32)
    return acc


def reduce_partials(partial: torch.Tensor, group=None, ordered: bool = True) -> torch.Tensor:
    """Layer output from this rank's partial output [M, d] (fp32), on every rank.

    ordered=True gathers the partial outputs and adds them in rank order (bitwise identical on every rank and
    from run to run); ordered=False is one all-reduce (what the benchmark times: NCCL over NVLink, [M, d] fp32
    is at most a few MB)."""
    import torch.distributed as dist
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return partial.to(torch.float32)
    if not ordered:
        out = partial.to(torch.float32).clone()
        dist.all_reduce(out, op=dist.ReduceOp.SUM, group=group)
        return out
    parts = [torch.empty_like(partial, dtype=torch.float32) for _ in range(dist.get_world_size(group))]
    dist.all_gather(parts, partial.to(torch.float32).contiguous(), group=group)
    return sum_in_rank_order(parts)
