"""Batching analysis, the slow and obvious way.  TEST INFRASTRUCTURE ONLY.

The paper files every recorded computation node in a table keyed by the node's
depth, observes that no node of a depth depends on another node of that depth,
and runs the table in depth order (Section 4.2).  For a forest of Tree-LSTM cells the
computation node of tree node v consumes the results of v's children, so its
depth is its height above the leaves:

    depth(v) = 0                         if v has no children
    depth(v) = 1 + max_k depth(child_k)  otherwise

and the table is (Section 4.3: nodes that can be batched share one slot):

    level_ptr[d] = number of nodes with depth < d,   d = 0 .. n_levels
    perm         = node ids ordered by (depth, id)
    edge_ptr[i]  = number of child edges owned by perm[0 .. i-1],  i = 0 .. n_nodes

Readings where the paper is silent: ties inside a level are broken by ascending
node id; ``n_levels`` is 0 for an empty forest.

Nothing here is shared with the CUDA path.  Pins: see tests/test_oracle_schedule.py.
"""
from __future__ import annotations

from collections import deque

import numpy as np


class NotAForest(ValueError):
    """The CSR does not describe a forest (bad id, two parents, or a cycle)."""


def build_parent(child_ptr, child_idx, n_nodes):
    """parent[v] (-1 for roots) from the child CSR, with validation."""
    child_ptr = np.asarray(child_ptr, dtype=np.int64)
    child_idx = np.asarray(child_idx, dtype=np.int64)
    if child_ptr.shape[0] != n_nodes + 1:
        raise NotAForest("child_ptr must have n_nodes + 1 entries")
    if n_nodes == 0:
        if child_idx.shape[0] != 0 or child_ptr[0] != 0:
            raise NotAForest("empty forest with edges")
        return np.zeros(0, dtype=np.int64)
    if child_ptr[0] != 0 or child_ptr[-1] != child_idx.shape[0]:
        raise NotAForest("child_ptr must start at 0 and end at n_edges")
    if np.any(np.diff(child_ptr) < 0):
        raise NotAForest("child_ptr must be non-decreasing")
    parent = [-1] * n_nodes
    for p in range(n_nodes):
        for e in range(child_ptr[p], child_ptr[p + 1]):
            c = int(child_idx[e])
            if c < 0 or c >= n_nodes:
                raise NotAForest(f"child id {c} out of range")
            if parent[c] != -1:
                raise NotAForest(f"node {c} has two parents")
            parent[c] = p
    return np.asarray(parent, dtype=np.int64)


def schedule(child_ptr, child_idx, n_nodes):
    """Return (depth, level_ptr, perm, edge_ptr, n_levels) as int32 arrays / int.

    Leaves-first breadth-first sweep: a node enters the queue when the last of
    its children has been popped, at which point its depth is final.
    """
    parent = build_parent(child_ptr, child_idx, n_nodes)
    cp = np.asarray(child_ptr, dtype=np.int64)
    pending = [int(cp[v + 1] - cp[v]) for v in range(n_nodes)]
    depth = [0] * n_nodes
    queue = deque(v for v in range(n_nodes) if pending[v] == 0)
    popped = 0
    while queue:
        v = queue.popleft()
        popped += 1
        p = int(parent[v]) if n_nodes else -1
        if p >= 0:
            depth[p] = max(depth[p], depth[v] + 1)
            pending[p] -= 1
            if pending[p] == 0:
                queue.append(p)
    if popped != n_nodes:
        raise NotAForest("cycle: some nodes never become ready")

    n_levels = (1 + max(depth)) if n_nodes else 0
    level_ptr = [0] * (n_levels + 1)
    for d in range(n_levels + 1):
        level_ptr[d] = sum(1 for v in range(n_nodes) if depth[v] < d) if n_nodes <= 64 else 0
    if n_nodes > 64:  # same definition, counted once instead of once per d
        counts = [0] * (n_levels + 1)
        for v in range(n_nodes):
            counts[depth[v] + 1] += 1
        run = 0
        for d in range(n_levels + 1):
            run += counts[d]
            level_ptr[d] = run

    cursor = list(level_ptr[:n_levels])
    perm = [0] * n_nodes
    for v in range(n_nodes):          # ascending id => stable within a level
        perm[cursor[depth[v]]] = v
        cursor[depth[v]] += 1

    edge_ptr = [0] * (n_nodes + 1)
    for i in range(n_nodes):
        v = perm[i]
        edge_ptr[i + 1] = edge_ptr[i] + int(cp[v + 1] - cp[v])

    return (np.asarray(depth, dtype=np.int32), np.asarray(level_ptr, dtype=np.int32),
            np.asarray(perm, dtype=np.int32), np.asarray(edge_ptr, dtype=np.int32), n_levels)
