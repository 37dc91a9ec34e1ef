"""Static draft-tree bookkeeping (oracle; test infrastructure).

Sec. 2.1: a static tree has a fixed shape; node 0 stands for the last committed
token, every other node carries one draft token, and the children of a node
are its s draft candidates in the order they were drawn.
"""


def tree_children(parent):
    """children[n] = list of child node ids of n in stored (rank) order.

    Requires breadth-first numbering: parent[0] = -1, parent[i] < i,
    parent[] non-decreasing (so children are contiguous)."""
    n = len(parent)
    if n < 1 or parent[0] != -1:
        raise ValueError("node 0 must be the root")
    children = [[] for _ in range(n)]
    for i in range(1, n):
        if not 0 <= parent[i] < i:
            raise ValueError("parent[i] must be in [0, i)")
        if parent[i] < parent[i - 1]:
            raise ValueError("nodes must be numbered breadth first")
        children[parent[i]].append(i)
    return children
