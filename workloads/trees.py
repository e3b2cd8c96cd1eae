"""Static candidate-tree templates and random tree topologies (inputs only).

A template lists, for every node, its parent, its depth and the top-k rank of
the draft head (depth d uses draft head d) whose candidate fills it.  Node 0 is
the root (the base head's own next token).  Nodes are ordered by (depth, rank
path), so "leftmost" means "smallest index" among nodes of one depth.

The paper builds its sparse trees from acceptance statistics on data that are
not available; the synthetic rule below only fixes *some* prefix-closed 64-node
subset of the top-10 tree with the right shape (more nodes on low ranks and
shallow depths).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class TreeTemplate:
    parent: np.ndarray      # int32 [N], parent[0] = -1
    depth: np.ndarray       # int32 [N]
    rank: np.ndarray        # int32 [N], rank[0] = 0 (unused)

    @property
    def n_nodes(self) -> int:
        return int(self.parent.shape[0])

    @property
    def max_depth(self) -> int:
        return int(self.depth.max())

    def rank_path(self, n: int) -> Tuple[int, ...]:
        out: List[int] = []
        while n > 0:
            out.append(int(self.rank[n]))
            n = int(self.parent[n])
        return tuple(reversed(out))

    def node_path(self, n: int) -> List[int]:
        out: List[int] = []
        while n >= 0:
            out.append(n)
            n = int(self.parent[n])
        return list(reversed(out))

    def leaves(self) -> List[int]:
        has_child = np.zeros(self.n_nodes, dtype=bool)
        has_child[self.parent[1:]] = True
        return [n for n in range(self.n_nodes) if not has_child[n]]

    def children(self, n: int) -> List[int]:
        return [m for m in range(1, self.n_nodes) if int(self.parent[m]) == n]


def _from_rank_paths(paths: Sequence[Tuple[int, ...]]) -> TreeTemplate:
    paths = sorted(set(paths), key=lambda p: (len(p), p))
    assert paths[0] == ()
    index = {p: i for i, p in enumerate(paths)}
    parent = np.array([-1] + [index[p[:-1]] for p in paths[1:]], dtype=np.int32)
    depth = np.array([len(p) for p in paths], dtype=np.int32)
    rank = np.array([0] + [p[-1] for p in paths[1:]], dtype=np.int32)
    return TreeTemplate(parent=parent, depth=depth, rank=rank)


def static_template(n_nodes: int, caps: Sequence[int]) -> TreeTemplate:
    """Root plus the n_nodes-1 cheapest rank paths under an integer cost.

    cost(path) = sum over edges j of (511 + 105*j + 357*rank_j), rank_j < caps[j];
    ties go to the shallower, then lexicographically smaller path.  The cost of a
    path exceeds that of each of its prefixes, so the choice is prefix-closed.
    """
    cand: List[Tuple[int, int, Tuple[int, ...]]] = []

    def grow(path: Tuple[int, ...], cost: int):
        j = len(path)
        if j == len(caps):
            return
        for r in range(caps[j]):
            c = cost + 511 + 105 * j + 357 * r
            p = path + (r,)
            cand.append((c, len(p), p))
            grow(p, c)

    grow((), 0)
    cand.sort()
    if n_nodes - 1 > len(cand):
        raise ValueError("template larger than the capped tree")
    chosen = [()] + [p for _, _, p in cand[: n_nodes - 1]]
    return _from_rank_paths(chosen)


def chain_template(n_nodes: int) -> TreeTemplate:
    """A path: node i is the only child of node i-1 (rank 0 everywhere)."""
    return TreeTemplate(parent=np.arange(-1, n_nodes - 1, dtype=np.int32),
                        depth=np.arange(n_nodes, dtype=np.int32),
                        rank=np.zeros(n_nodes, dtype=np.int32))


def random_topology(n_nodes: int, max_depth: int, seed: int) -> TreeTemplate:
    """Node n >= 1 picks a uniform parent among earlier nodes of depth < max_depth;
    the rank of a node is its order among its siblings; nodes are then re-indexed
    to (depth, rank path) order."""
    g = np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), 4]))
    parent = [-1]
    depth = [0]
    nchild = [0]
    paths: List[Tuple[int, ...]] = [()]
    for n in range(1, n_nodes):
        ok = [m for m in range(n) if depth[m] < max_depth]
        p = ok[int(g.integers(0, len(ok)))]
        parent.append(p)
        depth.append(depth[p] + 1)
        paths.append(paths[p] + (nchild[p],))
        nchild[p] += 1
        nchild.append(0)
    return _from_rank_paths(paths)


def depths_of(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int32)
    for n in range(1, len(parent)):
        d[n] = d[int(parent[n])] + 1
    return d


def ancestor_masks(parent: np.ndarray) -> np.ndarray:
    """Per node the bits of the node itself and all its ancestors: uint64 [n_nodes] for up to 64 nodes,
    uint64 [n_nodes][2] (bits 0..63, 64..127) for up to 128."""
    n_nodes = len(parent)
    if n_nodes > 128:
        raise ValueError("two 64-bit words hold at most 128 nodes")
    m = [0] * n_nodes
    for n in range(n_nodes):
        m[n] = (1 << n) | (m[int(parent[n])] if n > 0 else 0)
    if n_nodes <= 64:
        return np.array(m, dtype=np.uint64)
    return np.array([[x & (2**64 - 1), x >> 64] for x in m], dtype=np.uint64)


def validate_template(t: TreeTemplate, caps: Sequence[int] | None = None) -> None:
    """Raises ValueError unless the template is a rooted tree in (depth, rank path)
    order with distinct sibling ranks (and ranks below the caps, if given)."""
    n = t.n_nodes
    if n < 1 or t.parent[0] != -1 or t.depth[0] != 0:
        raise ValueError("node 0 must be the root")
    seen = set()
    prev_key = (0, ())
    for i in range(1, n):
        p = int(t.parent[i])
        if not (0 <= p < i):
            raise ValueError(f"node {i}: parent {p} must precede it")
        if t.depth[i] != t.depth[p] + 1:
            raise ValueError(f"node {i}: depth is not parent's depth + 1")
        if (p, int(t.rank[i])) in seen:
            raise ValueError(f"node {i}: duplicate rank among siblings")
        seen.add((p, int(t.rank[i])))
        if caps is not None:
            d = int(t.depth[i])
            if d > len(caps) or not (0 <= t.rank[i] < caps[d - 1]):
                raise ValueError(f"node {i}: rank or depth beyond the caps")
        key = (int(t.depth[i]), t.rank_path(i))
        if not key > prev_key:
            raise ValueError(f"node {i}: nodes are not in (depth, rank path) order")
        prev_key = key
