"""Reduction-dimension layout selection for a producer with several consumers (Section 3.2.2, "Global: layout
selections based on reduction dimension"), written out step by step.  Test infrastructure only.

The paper gives the rule in words: optimise the producer's layout for the first k reduction dimensions its consumers
require (k = number of memory dimensions with contiguous, index-free access); if the consumers require more, keep
several copies of the data, each in such a combined layout.  Readings taken where it is silent: "first" = most
demanded (summed consumer weight), ties to the dimension already nearer the contiguous end; inside a layout the most
demanded dimension is the contiguous one; dimensions that are not served keep their relative order."""
from __future__ import annotations


def select_layouts(ndim, reduction_dims, weights=None, k=1):
    """Returns (layouts, layout_of_consumer).  layouts[l] lists the producer dimensions from outermost to contiguous."""
    weights = [1] * len(reduction_dims) if weights is None else list(weights)
    demand = {}
    for rd, w in zip(reduction_dims, weights):
        if rd >= 0:
            demand[rd] = demand.get(rd, 0) + w
    # step 1: rank the demanded dimensions
    ranked = sorted(demand, key=lambda d: (-demand[d], -d))
    # step 2: cut the ranking into groups of k; each group is one stored copy of the tensor
    groups = [ranked[i:i + k] for i in range(0, len(ranked), k)] or [[]]
    layouts, where = [], {}
    for l, grp in enumerate(groups):
        outer = [d for d in range(ndim) if d not in grp]
        layouts.append(outer + grp[::-1])                # most demanded last = contiguous
        for d in grp:
            where[d] = l
    return layouts, [0 if rd < 0 else where[rd] for rd in reduction_dims]
