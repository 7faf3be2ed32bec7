"""Launch counts at kernel and at cell (subgraph) granularity, counted one node at a time.  TEST INFRASTRUCTURE ONLY.

Section 3 of the paper compares two granularities for batching a Tree-LSTM over a batch of trees and prints, in its
table of kernel and subgraph statistics, four counts: launches without and with batching, at operator ("kernel")
and at cell ("subgraph") granularity.  Its explanation of the gap: a cell is 33 operators, 4 of which take a
different form for every number of children; batching whole cells therefore only merges cells that agree in their
number of children, while batching operators merges the other 29 across all cells of a depth.

The paper gives the counts for its dataset only, not the counting rule, so the rule is this reading of that
paragraph (nodes are filed by depth as in Section 4.2; two launches can merge when they have the same depth and the
same signature):

    cells, no batching        one launch per node                                   N
    cells, batched            one launch per distinct (depth, number of children)   |{(depth(v), k(v))}|
    operators, no batching    33 launches per node                                  33 N
    operators, batched        per depth d: 29 shared launches, plus 4 for every     sum_d (29 + 4 |{k(v) : depth(v) = d}|)
                              distinct number of children met at that depth

and the batching ratio of a granularity is its unbatched count over its batched count.  (The table's own operator
count is 33.75 per cell, not 33; the text says 33 and nothing explains the difference, so 33 is used.)

Nothing here is shared with the CUDA path.  Pins: tests/test_oracle_granularity.py.
"""
from __future__ import annotations

OPS_PER_CELL = 33        # Section 3
OPS_DYNAMIC = 4          # of which depend on the number of children


def launch_counts(child_ptr, depth):
    """(cells_unbatched, cells_batched, ops_unbatched, ops_batched, n_levels) for a forest with the given depths."""
    n = len(child_ptr) - 1
    pairs = set()
    for v in range(n):
        pairs.add((int(depth[v]), int(child_ptr[v + 1]) - int(child_ptr[v])))
    levels = set(d for d, _ in pairs)
    ops_batched = 0
    for d in levels:
        kinds = sum(1 for (dd, _) in pairs if dd == d)
        ops_batched += (OPS_PER_CELL - OPS_DYNAMIC) + OPS_DYNAMIC * kinds
    return n, len(pairs), OPS_PER_CELL * n, ops_batched, len(levels)
