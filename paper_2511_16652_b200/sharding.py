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


def all_gather_packed_signs(local_signs, n_members: int, pack, unpack, group=None):
    """Exchange of pair signs in the base-3 packing of the paper's distributed framework: every rank packs the int8
    signs {-1,0,1} of its own pairs five to a byte (``pack``: tensor -> uint8 tensor), one all-gather moves
    ~ n_members / 10 bytes in total, and every rank unpacks (``unpack``: (uint8 tensor, count) -> int8 tensor) the full
    [n_members / 2] vector.  ``pack`` / ``unpack`` are the library's ``egr_fitness_pack3`` / ``egr_fitness_unpack3``."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return local_signs
    world = dist.get_world_size(group)
    counts = [member_range(n_members, world, r, True)[1] // 2 for r in range(world)]
    width = (max(counts) + 4) // 5
    mine = pack(local_signs)
    padded = torch.zeros(width, dtype=torch.uint8, device=mine.device)
    padded[: mine.numel()] = mine
    out = torch.empty(world * width, dtype=torch.uint8, device=mine.device)
    dist.all_gather_into_tensor(out, padded, group=group)
    parts = [unpack(out[r * width: r * width + (counts[r] + 4) // 5].contiguous(), counts[r]) for r in range(world) if counts[r]]
    return torch.cat(parts) if parts else local_signs
