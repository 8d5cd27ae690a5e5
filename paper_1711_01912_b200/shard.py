"""Candidate sharding across ranks (one process per GPU).

Candidates are independent, so the path shards without any data-path
collective: every rank holds the whole graph and its device tables and
evaluates a contiguous slice of the candidates.  The only communication is an
optional gather of the small per-candidate results (cp, load, memload, viol)
for a caller that wants them in one place; it runs over whatever backend the
process group was created with (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import Dict, List, Tuple


def candidate_slice(P: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous slice [j0, j1) of rank `rank`; sizes differ by at most one,
    the first P % world ranks get the longer slices."""
    if world < 1 or not (0 <= rank < world) or P < 0:
        raise ValueError("need world >= 1, 0 <= rank < world, P >= 0")
    base, extra = divmod(P, world)
    j0 = rank * base + min(rank, extra)
    return j0, j0 + base + (1 if rank < extra else 0)


def all_slices(P: int, world: int) -> List[Tuple[int, int]]:
    return [candidate_slice(P, world, r) for r in range(world)]


def gather_summaries(local: Dict[str, "torch.Tensor"], P: int, group=None) -> Dict[str, "torch.Tensor"]:
    """All-gather per-candidate results.  `local` maps a name to a tensor whose
    LAST dimension runs over this rank's candidates (cp: [p_r], load: [k, p_r]).
    Returns tensors whose last dimension is P, in global candidate order, on
    every rank."""
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    slices = all_slices(P, world)
    widest = max(j1 - j0 for j0, j1 in slices)
    out = {}
    for name, t in local.items():
        j0, j1 = slices[rank]
        if t.shape[-1] != j1 - j0:
            raise ValueError(f"{name}: last dimension {t.shape[-1]} is not this rank's slice length {j1 - j0}")
        pad = torch.zeros(t.shape[:-1] + (widest,), dtype=t.dtype, device=t.device)
        pad[..., : j1 - j0] = t
        parts = [torch.empty_like(pad) for _ in range(world)]
        dist.all_gather(parts, pad, group=group)
        out[name] = torch.cat([p[..., : b - a] for p, (a, b) in zip(parts, slices)], dim=-1)
    return out
