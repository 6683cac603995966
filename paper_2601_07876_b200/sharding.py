"""Partition of a parameter group over ranks (host logic only).

The NOVAK step has no cross-element term, so a group can be cut anywhere:
rank r owns a contiguous range of the flattened parameter space and runs
``novak_step`` on its own slices with its own state (state memory p/N per
rank).  Nothing is exchanged inside the step; ranks only have to take the same
number of steps so that lookahead synchronisations coincide.
"""
from __future__ import annotations


def partition_flat(numel, world: int, align: int = 64):
    """Splits tensors of ``numel[i]`` elements into ``world`` contiguous ranges
    of the flattened space with sizes equal up to ``align`` elements.

    Returns, per rank, a list of ``(tensor, start, stop)`` slices (element
    offsets inside the tensor, ``start < stop``).  Cut points fall on multiples
    of ``align`` elements of the flattened space, so a rank's slices of 256-byte
    aligned tensors stay 16-byte aligned whenever the tensors' sizes are
    multiples of 4.
    """
    if world < 1 or align < 1 or any(n <= 0 for n in numel):
        raise ValueError("bad partition arguments")
    total = sum(numel)
    units = -(-total // align)
    cuts = [min(total, (units * r // world) * align) for r in range(world)] + [total]
    out, t, base = [], 0, 0          # base = flat offset of tensor t
    for r in range(world):
        lo, hi = cuts[r], cuts[r + 1]
        slices = []
        while lo < hi:
            while base + numel[t] <= lo:
                base += numel[t]
                t += 1
            stop = min(hi, base + numel[t])
            slices.append((t, lo - base, stop - base))
            lo = stop
        out.append(slices)
    return out
