"""Expert-parallel sharding of the layer across GPUs (one process per GPU): host-side helpers.

Every rank holds the expert weights of a contiguous range of E / world experts, runs the router and TEAM's
selection on the full (replicated) rows -- routing is identical everywhere -- computes only its own experts, and
leaves its partial sums in y; the layer output is the sum over the ranks.  The one exchange on the data path is
therefore an all-reduce of the computed rows of y ([T, H] fp32: 32 KB on the SDAR-shaped step), which
`combine_partial_outputs` runs through torch.distributed (NCCL over NVLink on GPUs, gloo on CPU).  Rows that were
not computed (cached tokens) are left alone on every rank.
"""
import torch
import torch.distributed as dist


def expert_range(n_experts, rank, world):
    """[lo, hi) of the routed experts owned by `rank`."""
    if world < 1 or n_experts % world:
        raise ValueError("n_experts must be a multiple of the number of ranks")
    per = n_experts // world
    return rank * per, (rank + 1) * per


def shard_experts(t, n_experts, rank, world, per_expert_rows=1):
    """The slice of an expert-major tensor (or of a flat tile-major buffer with `per_expert_rows` leading elements
    per expert) that belongs to `rank`; a view, no copy."""
    lo, hi = expert_range(n_experts, rank, world)
    return t[lo * per_expert_rows:hi * per_expert_rows]


def combine_partial_outputs(y_partial, tok_class, y_out=None, group=None):
    """Sum of the ranks' partial layer outputs on the computed rows (tok_class != 0); other rows keep y_out's (or
    y_partial's) values.  Returns the combined tensor."""
    computed = (tok_class != 0).to(torch.bool)
    part = torch.where(computed[:, None], y_partial, torch.zeros_like(y_partial))
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(part, op=dist.ReduceOp.SUM, group=group)
    out = y_partial.clone() if y_out is None else y_out
    out[computed] = part[computed]
    return out
