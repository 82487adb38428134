"""Element partitioning across ranks.

Elements are independent, so the operators shard over the element index with the
small operator matrices replicated and no exchange step: every rank runs the same
single-GPU call on its own contiguous range.
"""
from __future__ import annotations


def shard_range(E: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous range [e0, e1) of a strong-scaling split of E elements: sizes differ
    by at most one and earlier ranks take the larger shares."""
    if world < 1 or not (0 <= rank < world) or E < 0:
        raise ValueError("need 0 <= rank < world and E >= 0")
    base, extra = divmod(E, world)
    e0 = rank * base + min(rank, extra)
    return e0, e0 + base + (1 if rank < extra else 0)


def weak_range(E_per_rank: int, rank: int, world: int) -> tuple[int, int]:
    """Range of global element indices rank ``rank`` owns when every rank holds
    ``E_per_rank`` elements (weak scaling): disjoint, contiguous, rank-ordered."""
    if world < 1 or not (0 <= rank < world) or E_per_rank < 0:
        raise ValueError("need 0 <= rank < world and E_per_rank >= 0")
    return rank * E_per_rank, (rank + 1) * E_per_rank
