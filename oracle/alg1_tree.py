"""Initial tree for the data-driven tree optimisation (paper App. A.1, Algorithm 1), written out plainly.

TEST INFRASTRUCTURE: the tests compare the library's tree builder with this.  Nodes are created level by
level; a node's child count depends on its depth, on its rank among its siblings (`order`) and on how many
children its parent has; the first node of every level gets at least three children.  The paper fixes the
outcome: 625 nodes, maximum depth 20.
"""
import math


def initial_tree(levels: int = 20):
    """Returns (parent, depth, order) lists in creation order (node 0 = root)."""
    parent, depth, order, n_children_of = [-1], [0], [0], [0]
    active = [0]
    for _ in range(levels):
        created = []
        for i, node in enumerate(active):
            d = depth[node]
            if d == 0:
                n = 8
            elif d == 1:
                n = max(8 - 2 * order[node], 1)
            else:
                siblings = n_children_of[parent[node]]
                n = math.ceil((siblings - 1) / (order[node] * 0.7 + 1))
                n = max(n, 2 if d in (2, 3) else 0)
            if i == 0:
                n = max(n, 3)
            n_children_of[node] = n
            for k in range(n):
                parent.append(node)
                depth.append(d + 1)
                order.append(k)
                n_children_of.append(0)
                created.append(len(parent) - 1)
        active = created
    return parent, depth, order
