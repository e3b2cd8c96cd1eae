"""Sparse candidate-tree construction (test infrastructure only).

Sec. II-D: within a fixed number of nodes the sparse tree should maximise the
expected accepted length; the tree is grown greedily, one node at a time, from
acceptance probabilities measured with the full tree.  Here the statistics are
conditional edge probabilities prob[j][r] = P(the rank-r candidate of draft head
j+1 is accepted | its parent is accepted), a node's acceptance probability is the
product along its root path, and the expected accepted length of a tree is
1 (the root) + the sum of its nodes' probabilities.

`greedy_tree` takes the steps in the paper's order: start from the root, and N-1
times add the candidate child of the current tree with the highest probability.
`best_tree_brute_force` is the definition written out: it enumerates every
prefix-closed node set of the given size.  Ties go to the shallower, then the
lexicographically smaller rank path.
"""
from __future__ import annotations

import itertools
from typing import Dict, List, Sequence, Tuple

import numpy as np

Path = Tuple[int, ...]


def path_probability(prob: np.ndarray, path: Path) -> float:
    p = 1.0
    for j, r in enumerate(path):
        p *= float(prob[j][r])
    return p


def expected_length(prob: np.ndarray, paths: Sequence[Path]) -> float:
    """1 for the root plus the acceptance probability of every other node."""
    return 1.0 + sum(path_probability(prob, p) for p in paths if len(p) > 0)


def greedy_tree(prob: np.ndarray, n_nodes: int) -> List[Path]:
    depth, topk = prob.shape
    tree: List[Path] = [()]
    for _ in range(n_nodes - 1):
        in_tree = set(tree)
        best = None
        for parent in tree:
            if len(parent) == depth:
                continue
            for r in range(topk):
                c = parent + (r,)
                if c in in_tree:
                    continue
                key = (-path_probability(prob, c), len(c), c)
                if best is None or key < best[0]:
                    best = (key, c)
        if best is None:
            raise ValueError("the capped tree has fewer nodes than asked for")
        tree.append(best[1])
    return sorted(tree, key=lambda p: (len(p), p))


def best_tree_brute_force(prob: np.ndarray, n_nodes: int) -> Tuple[float, List[List[Path]]]:
    """(best expected length, all prefix-closed node sets of that size reaching it)."""
    depth, topk = prob.shape
    all_paths: List[Path] = []
    for d in range(1, depth + 1):
        all_paths += list(itertools.product(range(topk), repeat=d))
    best, arg = -1.0, []
    for subset in itertools.combinations(all_paths, n_nodes - 1):
        s = set(subset)
        if any(len(p) > 1 and p[:-1] not in s for p in subset):
            continue
        e = expected_length(prob, subset)
        if e > best + 1e-15:
            best, arg = e, [sorted([()] + list(subset), key=lambda p: (len(p), p))]
        elif abs(e - best) <= 1e-15:
            arg.append(sorted([()] + list(subset), key=lambda p: (len(p), p)))
    return best, arg


def to_arrays(paths: Sequence[Path]) -> Tuple[np.ndarray, np.ndarray]:
    """parent[] and rank[] of a node list in (depth, rank path) order."""
    paths = sorted(paths, key=lambda p: (len(p), p))
    index: Dict[Path, int] = {p: i for i, p in enumerate(paths)}
    parent = np.array([-1] + [index[p[:-1]] for p in paths[1:]], dtype=np.int32)
    rank = np.array([0] + [p[-1] for p in paths[1:]], dtype=np.int32)
    return parent, rank
