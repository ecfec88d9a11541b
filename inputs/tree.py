"""Seeded synthetic draft-tree topologies.

The paper's 64-node tree (Appendix A.1) was fitted on an auxiliary dataset and is
not printed, so a synthetic stand-in with the same structure is generated here: a
sparse tree of depth <= K whose level-k nodes name ranks in head k's top-k list,
chosen to maximise a synthetic acceptance score.  Only topology (parent / depth /
rank per node) is produced; ancestor masks, positions and path tables are derived
separately by the oracle and by the CUDA library.
"""
from __future__ import annotations

import heapq
from dataclasses import dataclass
from typing import List, Sequence, Tuple

from .gen import uniform_floats


@dataclass(frozen=True)
class TreeTopology:
    parent: Tuple[int, ...]   # parent[0] = -1 (root)
    depth: Tuple[int, ...]    # depth[0] = 0; depth k >= 1 means "head k"
    rank: Tuple[int, ...]     # rank within head depth[n]'s top-k list; rank[0] = 0

    @property
    def n_nodes(self) -> int:
        return len(self.parent)

    @property
    def max_depth(self) -> int:
        return max(self.depth)

    def widths(self) -> List[int]:
        """1 + the largest rank used at each depth 1..max_depth."""
        w = [0] * self.max_depth
        for n in range(1, self.n_nodes):
            w[self.depth[n] - 1] = max(w[self.depth[n] - 1], self.rank[n] + 1)
        return w


def _from_paths(paths: Sequence[Tuple[int, ...]]) -> TreeTopology:
    paths = sorted(set(paths), key=lambda p: (len(p), p))
    index = {(): 0}
    parent, depth, rank = [-1], [0], [0]
    for p in paths:
        assert p[:-1] in index, "tree must be prefix-closed"
        index[p] = len(parent)
        parent.append(index[p[:-1]])
        depth.append(len(p))
        rank.append(p[-1])
    return TreeTopology(tuple(parent), tuple(depth), tuple(rank))


def make_tree(n_nodes: int, widths: Sequence[int], seed: int = 2) -> TreeTopology:
    """Best-first tree of `n_nodes` (root included) under a synthetic rank-acceptance table.

    q[k][r] = A_k * 2^-(r+1) * jitter, A = (0.80, 0.65, 0.55, 0.45, ...), jitter ~ U(0.9, 1.1);
    a path's score is the product of q along it; the n_nodes-1 best paths are kept.
    Rows of q are made strictly decreasing in r so the result is sibling-closed.
    """
    K = len(widths)
    A = [0.80, 0.65, 0.55, 0.45] + [0.40] * max(0, K - 4)
    u = uniform_floats(K * 16, seed, "tree_jitter")
    q: List[List[float]] = []
    for k in range(K):
        row: List[float] = []
        for r in range(widths[k]):
            v = A[k] * 2.0 ** (-(r + 1)) * (0.9 + 0.2 * u[k * 16 + (r % 16)])
            if row and v >= row[-1]:
                v = row[-1] * 0.999
            row.append(v)
        q.append(row)
    heap: List[Tuple[float, int, Tuple[int, ...]]] = []
    if K and widths[0] > 0:
        heapq.heappush(heap, (-q[0][0], 1, (0,)))
    chosen: List[Tuple[int, ...]] = []
    score = {(0,): q[0][0]} if K and widths[0] > 0 else {}
    while heap and len(chosen) < n_nodes - 1:
        negs, d, p = heapq.heappop(heap)
        chosen.append(p)
        s = -negs
        if d < K and widths[d] > 0:                       # first child
            c = p + (0,)
            score[c] = s * q[d][0]
            heapq.heappush(heap, (-score[c], d + 1, c))
        r = p[-1]
        if r + 1 < widths[d - 1]:                         # next sibling
            sib = p[:-1] + (r + 1,)
            score[sib] = s / q[d - 1][r] * q[d - 1][r + 1]
            heapq.heappush(heap, (-score[sib], d, sib))
    return _from_paths(chosen)


def full_tree(widths: Sequence[int]) -> TreeTopology:
    """Every combination of ranks: level k has prod(widths[:k]) nodes (Fig. 5's example)."""
    paths: List[Tuple[int, ...]] = []
    level: List[Tuple[int, ...]] = [()]
    for w in widths:
        level = [p + (r,) for p in level for r in range(w)]
        paths += level
    return _from_paths(paths)


def chain_tree(n_nodes: int) -> TreeTopology:
    """A path: node i's parent is i-1, every rank 0."""
    return _from_paths([(0,) * k for k in range(1, n_nodes)])
