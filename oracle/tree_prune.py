"""Selection half of the data-driven tree optimisation (paper Sec. 4.2), written out plainly.

TEST INFRASTRUCTURE.  The nodes of a large tree are ranked by how often they were accepted and the top
`keep` form the new tree (the paper keeps the top 80 of 625).  Equal counts go to the lower index.
"""


def prune_tree(parent, counts, keep):
    """Returns (new_parent, old_index): the tree of the `keep` most accepted nodes, renumbered in the old order."""
    order = sorted(range(len(parent)), key=lambda u: (-int(counts[u]), u))
    kept = sorted(order[:keep])
    new_index = {u: i for i, u in enumerate(kept)}
    new_parent = [-1 if parent[u] < 0 else new_index[parent[u]] for u in kept]
    return new_parent, kept
