"""Synthetic draft trees of an exact size, for exercising tree attention and acceptance on their own.

The drafter's real trees depend on the table contents; these stand-ins have exactly ``n`` nodes with
seeded random parents under a depth cap, parents always preceding children (the order a breadth-first
drafter emits).  The bit-packed ancestor relation is produced here only as an *input* for attention-only
cases; the drafter's own mask output is checked separately.
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


def tree_mask_from_parents(par: np.ndarray, n: int, words: int) -> np.ndarray:
    """uint32 [T, words]: bit j of row i set iff node j is node i or one of its ancestors; rows >= n zero."""
    T = par.shape[0]
    m = np.zeros((T, words), dtype=np.uint32)
    for i in range(n):
        if par[i] >= 0:
            m[i] = m[par[i]]
        m[i, i // 32] |= np.uint32(1) << np.uint32(i % 32)
    return m
