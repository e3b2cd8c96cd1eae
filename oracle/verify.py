"""Verification with the tolerance mechanism (Algorithm 1) and the choice among
branches (Sec. II-C).  Test infrastructure only.

`verify_branch` + `select_best` are the defining routines: one branch at a time,
then longest accepted sequence, then leftmost.  `tree_edge_accepts` +
`accept_from_edges` state the same decision once for the whole tree (one test
per edge, one ancestor walk per node); they exist to be checked against the
per-branch routines by brute force.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def verify_branch(cands: Sequence[int], sets: Sequence[Sequence[int]]) -> int:
    """Tolerance check of one branch (Algorithm 1, Sec. II-C), after the draw sets have been made.

    cands = (c_0, ..., c_k) are the branch's tokens from the root down; sets[i] holds
    the tau tokens the base head drew at c_i.  The root is the base head's own token and
    is always kept; the accepted part of the branch ends just before the first child
    that is missing from its parent's draws.  Returns the index of the last accepted
    candidate (so that many + 1 tokens are accepted)."""
    misses = [i for i in range(len(cands) - 1) if cands[i + 1] not in sets[i]]
    return misses[0] if misses else len(cands) - 1


def select_best(branches: Sequence[Tuple[Tuple[int, ...], int]]) -> int:
    """Index of the winning branch.

    branches[i] = (rank path of branch i, k*_i).  The longest accepted sequence
    wins; among equally long ones the leftmost, i.e. the one whose accepted part
    uses the smallest top-k ranks, compared from the root down."""
    best, best_key = -1, None
    for i, (ranks, k_star) in enumerate(branches):
        key = (-k_star, tuple(ranks[:k_star]))
        if best_key is None or key < best_key:
            best, best_key = i, key
    return best


def tree_edge_accepts(parent: np.ndarray, tokens: np.ndarray, sets_per_node) -> np.ndarray:
    """edge_ok[n] for n >= 1: the token of node n is among the draws made at its
    parent.  edge_ok[0] is True (the root is the base head's own token)."""
    n_nodes = len(parent)
    ok = np.zeros(n_nodes, dtype=bool)
    ok[0] = True
    for n in range(1, n_nodes):
        ok[n] = int(tokens[n]) in sets_per_node[int(parent[n])]
    return ok


def accept_from_edges(parent: np.ndarray, depth: np.ndarray, edge_ok: np.ndarray) -> Tuple[int, List[int]]:
    """Whole-tree form of the decision: a node is accepted when every edge from
    the root down to it is; the winner is the deepest accepted node, the one
    with the smallest index among equally deep ones (nodes are stored in
    (depth, rank path) order).  Returns (winner, its root path)."""
    n_nodes = len(parent)
    acc = np.zeros(n_nodes, dtype=bool)
    acc[0] = True
    for n in range(1, n_nodes):
        acc[n] = acc[int(parent[n])] and bool(edge_ok[n])
    best = 0
    for n in range(n_nodes):
        if acc[n] and depth[n] > depth[best]:
            best = n
    path = []
    n = best
    while n >= 0:
        path.append(n)
        n = int(parent[n])
    return best, path[::-1]
