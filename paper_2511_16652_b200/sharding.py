"""Population sharding over GPUs (Algorithm 1: "workers share scalar fitness f_i with other workers", then every
worker rebuilds all E_j from the seeds and applies the same update).

Members are split into contiguous ranges, one per rank (antithetic pairs are never split).  A rank evaluates its
own members with ``Layer(member_base=...)``, the ranks exchange N scalars with one all-gather, and every rank applies
the identical full update locally: no weight traffic at all.  Only plumbing lives here; the arithmetic stays in the
kernels behind the C ABI.
"""
from __future__ import annotations


def member_range(n_members: int, world: int, rank: int, antithetic: bool = False):
    """(first member, member count) of ``rank``: contiguous, balanced to within one unit, pairs kept together."""
    unit = 2 if antithetic else 1
    if n_members % unit:
        raise ValueError("an antithetic population has an even number of members")
    units = n_members // unit
    lo = units * rank // world
    hi = units * (rank + 1) // world
    return lo * unit, (hi - lo) * unit


def all_gather_fitness(local, n_members: int, antithetic: bool = False, group=None):
    """Concatenate every rank's raw fitness (1-D tensor of its member range) into the full [n_members] vector.

    Ranges may differ in length by one unit, so shorter ones are padded for the collective and trimmed afterwards."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return local
    world = dist.get_world_size(group)
    counts = [member_range(n_members, world, r, antithetic)[1] for r in range(world)]
    width = max(counts)
    padded = torch.zeros(width, dtype=local.dtype, device=local.device)
    padded[: local.numel()] = local
    out = torch.empty(world * width, dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(out, padded, group=group)
    return torch.cat([out[r * width: r * width + counts[r]] for r in range(world)])
