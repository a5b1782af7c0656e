"""Column shards of the parameter matrix for the mix on several GPUs.

The update of Eqs. 4-5 (and Eq. 3) acts on every column of the N x d parameter matrix independently: column c
of X' depends on column c of X and G and on the weights only.  So rank r of R can own the columns [c0_r, c1_r)
of X, G and X' as an N x (c1_r - c0_r) matrix of its own, run the same round on it (its own dbw_init with
d = c1_r - c0_r; selection, weights and times are replicated, they cost microseconds), and no data ever crosses
between ranks.  This module only computes the partition; it holds none of the method's arithmetic.
"""
from __future__ import annotations

from typing import List, Tuple


def column_shards(d: int, world: int, align: int = 4) -> List[Tuple[int, int]]:
    """[(c0, c1)] for ranks 0 .. world-1: contiguous, disjoint, covering [0, d), every inner boundary a multiple of
    `align` columns (4 floats = the 16-byte alignment the kernels' 128-bit loads need), widths equal up to `align`."""
    if d < 1 or world < 1 or align < 1:
        raise ValueError("d, world and align must be positive")
    units = (d + align - 1) // align
    if world > units:
        raise ValueError("more ranks than %d-column units" % align)
    bounds = [min(d, align * ((units * r) // world)) for r in range(world)] + [d]
    return [(bounds[r], bounds[r + 1]) for r in range(world)]
