"""Synthetic draft trees of an exact size, for exercising tree attention and acceptance on their own.

The drafter's real trees depend on the table contents; these stand-ins have exactly ``n`` nodes with
seeded random parents under a depth cap, parents always preceding children (the order a breadth-first
drafter emits).  Only parents and depths are produced here; the ancestor masks that attention-only cases
need as an input are made by their callers.
"""
import numpy as np

from .rng import mix64

_TID_TREE = 201


def random_tree(seed: int, b: int, n: int, max_depth: int, max_nodes: int = None):
    """Returns (parent int32 [T], depth int32 [T]) padded with -1 to T = max_nodes (default n)."""
    T = n if max_nodes is None else max_nodes
    par = np.full(T, -1, dtype=np.int32)
    dep = np.full(T, -1, dtype=np.int32)
    if n > 0:
        dep[0] = 0
    h = mix64(seed, _TID_TREE, b * 4096 + np.arange(max(n, 1)))
    for i in range(1, n):
        cand = [j for j in range(i) if dep[j] < max_depth]
        # bias towards recent nodes so that trees get deep as well as wide
        pick = int(h[i] % np.uint64(len(cand)))
        if (int(h[i]) >> 40) & 1:
            pick = len(cand) - 1 - (pick % min(len(cand), 3))
        par[i] = cand[pick]
        dep[i] = dep[par[i]] + 1
    return par, dep
