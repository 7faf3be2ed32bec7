"""Pins for the launch-count checker (oracle/granularity.py): hand-counted forests and closed forms."""
import numpy as np

from conftest import read_golden
from oracle import granularity as og
from oracle import schedule as osched
from paper_1904_07421_b200 import workloads as wl


def counts(forest):
    depth = osched.schedule(forest.child_ptr, forest.child_idx, forest.n_nodes)[0]
    return og.launch_counts(forest.child_ptr, depth)


def test_hand_counted_forest():
    g = read_golden("forest10.txt")
    assert list(og.launch_counts(g["child_ptr"], g["depth"])) == g["launch_counts"]


def test_two_kinds_of_cell_on_one_level_by_hand():
    # 0 -> (1, 2, 3); 1 -> (4); 2 -> (5, 6): depth 1 holds a one-child and a two-child cell
    f = wl.forest_from_parents([np.array([-1, 0, 0, 0, 1, 2, 2])])
    # pairs (0,0), (1,1), (1,2), (2,3); operators: (29 + 4) + (29 + 8) + (29 + 4)
    assert counts(f) == (7, 4, 231, 103, 3)


def test_chain_star_and_complete_binary_tree():
    n = 17
    chain = wl.forest_from_parents([np.array([-1] + list(range(n - 1)))])
    assert counts(chain) == (n, n, 33 * n, 33 * n, n)            # nothing to batch: one cell per depth
    star = wl.forest_from_parents([np.array([-1] + [0] * (n - 1))])
    assert counts(star) == (n, 2, 33 * n, 66, 2)
    h = 5
    parent = np.array([-1] + [(i - 1) // 2 for i in range(1, 2 ** (h + 1) - 1)])
    tree = wl.forest_from_parents([parent])
    assert counts(tree) == (2 ** (h + 1) - 1, h + 1, 33 * (2 ** (h + 1) - 1), 33 * (h + 1), h + 1)


def test_copies_batch_for_free_and_labels_do_not_matter():
    w = wl.make_workload(1, n_trees=9)
    one = counts(w.forest)
    parents = [wl.parent_array(wl.subforest(w.forest, [t])[0]) for t in range(9)]
    three = counts(wl.forest_from_parents(parents * 3))
    assert three[0] == 3 * one[0] and three[2] == 3 * one[2]     # unbatched counts grow with the batch ...
    assert three[1] == one[1] and three[3] == one[3]             # ... batched ones do not
    g, _ = wl.relabel(w.forest, np.random.default_rng(4))
    assert counts(g) == one
    # operator batching never needs more launches than 33 per batched cell, and is at least 33 per level
    assert 33 * one[4] <= one[3] <= 33 * one[1]
