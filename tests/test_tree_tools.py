"""Static-tree tools: Algorithm 1's initial tree and the acceptance-frequency pruning (paper Sec. 4.2, App. A.1)."""
import collections

import numpy as np
import pytest

from oracle import alg1_tree, tree_prune
from paper_2506_04708_b200 import binding, build as lib_build, inputs


@pytest.fixture(scope="module", autouse=True)
def _lib():
    lib_build.build()


def test_oracle_tree_has_the_size_the_paper_states():
    # App. A.1: "the resulting tree has a maximum depth of 20 and 625 total nodes"
    parent, depth, order = alg1_tree.initial_tree()
    assert len(parent) == 625 and max(depth) == 20
    # what the rules fix directly: 8 children of the root, max(8 - 2 * order, 1) below (the first node >= 3)
    kids = collections.Counter(parent[1:])
    assert kids[0] == 8
    assert [kids[u] for u in range(1, 9)] == [8, 6, 4, 2, 1, 1, 1, 1]
    # the long tail of the paper's figure: one chain of width max(ceil((w - 1) / 1), 3) = 8 at the deep levels
    per_depth = collections.Counter(depth)
    assert [per_depth[d] for d in range(9, 21)] == [8] * 12


def test_library_tree_equals_the_oracle_tree():
    parent, depth, order, total = binding.initial_tree()
    o_parent, o_depth, o_order = alg1_tree.initial_tree()
    assert total == 625
    assert parent.tolist() == o_parent and depth.tolist() == o_depth and order.tolist() == o_order
    for levels in (0, 1, 2, 5, 9):
        p, d, o, t = binding.initial_tree(levels)
        op, od, oo = alg1_tree.initial_tree(levels)
        assert t == len(op) and p.tolist() == op and d.tolist() == od
    # a prefix in creation order is a valid topology for the library (parents first, siblings together)
    p128, _, _, t = binding.initial_tree(20, capacity=128)
    assert t == 625 and len(p128) == 128 and p128.tolist() == o_parent[:128]
    cfg = binding.make_config(1, 128, 1000, 8, 3, 0, 1.0, 0, 1 << 10, p128)
    assert binding.workspace_bytes(cfg) > 0


def test_prune_keeps_the_most_accepted_nodes():
    parent = inputs.topology(24, 6, 3)
    rng = np.random.default_rng(3)
    # acceptance counts: never larger than the parent's
    counts = np.zeros(len(parent), np.uint64)
    counts[0] = 1000
    for u in range(1, len(parent)):
        counts[u] = rng.integers(0, int(counts[parent[u]]) + 1)
    for keep in (1, 2, 7, 16, 24):
        got_parent, got_old = binding.prune_tree(parent, counts, keep)
        want_parent, want_old = tree_prune.prune_tree(parent.tolist(), counts.tolist(), keep)
        assert got_parent.tolist() == want_parent and got_old.tolist() == want_old
        # still a valid topology
        cfg = binding.make_config(1, keep, 1000, 8, 3, 0, 1.0, 0, 1 << 10, got_parent)
        assert binding.workspace_bytes(cfg) > 0
    # ties go to the lower index; invalid requests are refused
    flat = np.full(len(parent), 5, np.uint64)
    p2, old = binding.prune_tree(parent, flat, 4)
    assert old.tolist() == [0, 1, 2, 3]
    with pytest.raises(binding.StandError):
        binding.prune_tree(parent, counts, 0)
    with pytest.raises(binding.StandError):
        binding.prune_tree(parent, counts, 25)
    bad = counts.copy()
    bad[0] = 0  # the root ranked out: not acceptance counts
    with pytest.raises(binding.StandError):
        binding.prune_tree(parent, bad, 3)
