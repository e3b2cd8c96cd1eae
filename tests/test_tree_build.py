"""Sparse-tree construction (paper Sec. II-D): the oracle's greedy growth against the definition (exhaustive
search for the largest expected accepted length), and the library's host routine against the oracle."""
import numpy as np
import pytest

import oracle as O
import workloads as W
from oracle import tree_build as T


def _probs(seed, depth, topk, sorted_ranks):
    g = np.random.Generator(np.random.Philox(key=[seed, 77]))
    p = g.uniform(0.02, 0.9, size=(depth, topk))
    return -np.sort(-p, axis=1) if sorted_ranks else p


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("sorted_ranks", [True, False])
def test_greedy_growth_reaches_the_exhaustive_optimum(seed, sorted_ranks):
    prob = _probs(seed, 3, 3, sorted_ranks)
    for n in (1, 2, 4, 6, 7):
        tree = O.greedy_tree(prob, n)
        best, arg = O.best_tree_brute_force(prob, n)
        assert abs(O.expected_length(prob, tree) - best) < 1e-12
        assert tree in arg
        assert tree[0] == () and all(p[:-1] in tree for p in tree[1:])        # prefix-closed


def test_closed_forms():
    # one head, probabilities q_r: the tree is the n-1 best ranks, expected length 1 + their sum
    prob = np.array([[0.5, 0.3, 0.1, 0.05]])
    tree = O.greedy_tree(prob, 3)
    assert tree == [(), (0,), (1,)] and abs(O.expected_length(prob, tree) - 1.8) < 1e-15
    # a single candidate per head with probability q: a chain, expected length 1 + q + q^2 + ...
    prob = np.full((4, 1), 0.5)
    tree = O.greedy_tree(prob, 5)
    assert tree == [(), (0,), (0, 0), (0, 0, 0), (0, 0, 0, 0)]
    assert abs(O.expected_length(prob, tree) - (1 + 0.5 + 0.25 + 0.125 + 0.0625)) < 1e-15
    with pytest.raises(ValueError):
        O.greedy_tree(prob, 6)
    # ties: shallower first, then the smaller rank path
    prob = np.full((2, 2), 0.5)
    assert O.greedy_tree(prob, 4) == [(), (0,), (1,), (0, 0)]


@pytest.mark.parametrize("seed,depth,topk,n", [(1, 3, 3, 7), (2, 4, 10, 64), (3, 6, 10, 64), (4, 4, 5, 42), (5, 2, 2, 7)])
def test_library_routine_equals_the_oracle(seed, depth, topk, n):
    import paper_2410_21951_b200 as P
    prob = _probs(seed, depth, topk, sorted_ranks=(seed % 2 == 0))
    parent, rank, exp = P.build_sparse_tree(prob, n)
    want = O.greedy_tree(prob, n)
    wp, wr = T.to_arrays(want)
    assert np.array_equal(parent, wp) and np.array_equal(rank, wr)
    assert abs(exp - O.expected_length(prob, want)) < 1e-12
    tpl = W.TreeTemplate(parent=parent, depth=W.depths_of(parent), rank=rank) if hasattr(W, "TreeTemplate") else None
    if tpl is not None:
        W.validate_template(tpl, [topk] * depth)


def test_library_routine_rejects_bad_requests():
    import paper_2410_21951_b200 as P
    with pytest.raises(P.VadusaError):
        P.build_sparse_tree(np.full((1, 2), 0.5), 4)          # only 3 nodes exist
    with pytest.raises(P.VadusaError):
        P.build_sparse_tree(np.full((16, 2), 0.5), 4)         # deeper than the library's limit
