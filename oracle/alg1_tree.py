"""Initial tree for the data-driven tree optimisation (paper App. A.1, Algorithm 1), as a definition by paths.

TEST INFRASTRUCTURE: the tests compare the library's tree builder with this.

A node is named by the sibling ranks on the way down from the root: () is the root, (0, 2) the third child of
the root's first child.  App. A.1's rules make the number of children a function of that name alone:

    width(())          = 8
    width((r,))        = max(8 - 2 r, 1)
    width(path + (r,)) = max(ceil((width(path) - 1) / (0.7 r + 1)), 2 at depths 2 and 3, else 0)

and the leftmost node of every level, the all-zero path, has at least three children.  The tree is the set of
paths whose every rank is below the width of the prefix before it; creation order (level by level, parents in
order, children by rank) is the order of (depth, path).  The paper fixes the outcome: 625 nodes, depth 20.
"""
import functools
import math


@functools.lru_cache(maxsize=None)
def width(path):
    """Children of the node with this path of sibling ranks."""
    depth = len(path)
    if depth == 0:
        n = 8
    elif depth == 1:
        n = max(8 - 2 * path[-1], 1)
    else:
        n = max(math.ceil((width(path[:-1]) - 1) / (0.7 * path[-1] + 1)), 2 if depth in (2, 3) else 0)
    return max(n, 3) if not any(path) else n


def initial_tree(levels: int = 20):
    """Returns (parent, depth, order) lists in creation order (node 0 = root)."""
    level = [()]
    paths = [()]
    for _ in range(levels):
        level = [p + (r,) for p in level for r in range(width(p))]  # already in (path) order
        paths += level
    index = {p: i for i, p in enumerate(paths)}
    parent = [-1] + [index[p[:-1]] for p in paths[1:]]
    depth = [len(p) for p in paths]
    order = [p[-1] if p else 0 for p in paths]
    return parent, depth, order
