"""How the path spreads over several GPUs: every (batch, head) pair is an
independent unit with the same plan, so ranks take disjoint contiguous slices
of the batch*heads axis and never exchange data (no collective in the path)."""
from __future__ import annotations


def unit_slice(n_units: int, world: int, rank: int) -> tuple[int, int]:
    """[begin, end) of the (batch*heads) units rank `rank` owns; sizes differ by at most one."""
    if world < 1 or not 0 <= rank < world or n_units < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(n_units, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)
