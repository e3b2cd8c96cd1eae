"""Pins of the oracle's sampler: the published splitmix64 vectors, the closed
forms of the Gumbel construction, and brute-force set membership."""
import itertools
import json
import os

import numpy as np

import oracle as O
from oracle import sampling as S

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_splitmix64_published_vectors():
    v = json.load(open(os.path.join(GOLDEN, "splitmix64_vectors.json")))
    state = v["seed"]
    for expect in v["outputs_hex"]:
        state = (state + S._GOLDEN) & S._M64
        assert S._mix_int(state) == int(expect, 16)
    arr = S._mix_arr(np.array([(S._GOLDEN * k) & S._M64 for k in range(1, 5)], dtype=np.uint64))
    assert [int(a) for a in arr] == [int(e, 16) for e in v["outputs_hex"]]


def test_uniform_is_exact_open_interval_and_keyed_by_all_fields():
    u = O.uniform23(1, 0, 5, 4096)
    assert u.dtype == np.float32 and u.min() > 0.0 and u.max() < 1.0
    x = u.astype(np.float64) * 2 ** 23 - 0.5
    assert np.array_equal(x, np.round(x)) and x.min() >= 0 and x.max() < 2 ** 23
    base = O.uniform23(1, 0, 5, 64)
    for other in (O.uniform23(2, 0, 5, 64), O.uniform23(1, 1, 5, 64), O.uniform23(1, 0, 6, 64)):
        assert np.mean(other == base) < 0.1
    assert abs(O.uniform23(3, 2, 9, 200000).mean() - 0.5) < 0.005


def test_gumbel_mean_is_euler_gamma_and_variance_pi2_over_6():
    g = np.concatenate([O.gumbel_noise(11, s, 3, 50000) for s in range(8)]).astype(np.float64)
    assert abs(g.mean() - 0.5772156649) < 0.01
    assert abs(g.var() - np.pi ** 2 / 6) < 0.03


def test_first_draw_frequencies_match_softmax():
    """Gumbel-arg-max draws token j with probability softmax(logits / T)_j."""
    g = np.random.default_rng(3)
    V, T, trials = 16, 0.8, 40000
    logits = g.standard_normal(V) * 1.5
    l32 = logits.astype(np.float32)
    p = np.exp(logits / T); p /= p.sum()
    counts = np.zeros(V)
    nuc = np.ones(V, dtype=bool)
    for pos in range(trials):
        counts[O.root_token(O.decision_keys(l32, T, 5, 0, pos), nuc)] += 1
    chi2 = ((counts - trials * p) ** 2 / (trials * p)).sum()
    assert chi2 < 45.0          # 15 degrees of freedom; P(chi2 > 45) < 1e-4
    # and the pair (first, second) follows sampling without replacement
    pair = np.zeros((V, V))
    for pos in range(trials):
        a, b = O.sample_set(O.decision_keys(l32, T, 6, 0, pos), nuc, 2)
        pair[a, b] += 1
    expect = trials * p[:, None] * p[None, :] / (1 - p[:, None])
    np.fill_diagonal(expect, 0)
    assert np.trace(pair) == 0
    big = expect > 20
    assert (((pair - expect) ** 2)[big] / expect[big]).sum() < big.sum() + 6 * np.sqrt(2 * big.sum())


def test_greedy_keys_are_the_logits_and_eos_is_masked():
    l = np.array([0.1, 2.0, -1.0, 5.0])
    l32 = S.masked_logits32(l, eos_id=3, eos_masked=True)
    assert l32[3] == -np.inf
    keys = O.decision_keys(l32, 0.0, 1, 0, 0)
    nuc = O.nucleus_sorted(l32, 0.0, 0.5)
    assert O.sample_set(keys, nuc, 3) == [1, 0, 2] and not nuc[3]


def test_nucleus_by_sorting_brute_force():
    """Shortest descending-probability prefix whose mass reaches top_p, against
    an enumeration of all prefixes."""
    g = np.random.default_rng(4)
    for _ in range(200):
        V = int(g.integers(2, 9))
        l32 = (g.standard_normal(V) * 2).astype(np.float32)
        if g.random() < 0.3:
            l32[int(g.integers(0, V))] = l32[0]                    # ties
        T = float(g.choice([0.5, 1.0, 1.3])); top_p = float(g.uniform(0.05, 0.999))
        p = np.exp(l32.astype(np.float64) / T); p /= p.sum()
        order = sorted(range(V), key=lambda j: (-p[j], j))
        size = next(k for k in range(1, V + 1) if sum(p[j] for j in order[:k]) >= top_p or k == V)
        expect = np.zeros(V, dtype=bool); expect[order[:size]] = True
        assert np.array_equal(O.nucleus_sorted(l32, T, top_p), expect)
        for c in range(V):
            assert (O.nucleus_mass_before(l32, T, c) < top_p) == expect[c]


def test_rank_count_membership_equals_sorted_membership():
    g = np.random.default_rng(5)
    # exhaustive over small key patterns with ties
    for V in (3, 4, 5):
        for pattern in itertools.product(range(3), repeat=V):
            keys = np.array(pattern, dtype=np.float32)
            for nucbits in range(1, 2 ** V):
                nuc = np.array([(nucbits >> j) & 1 for j in range(V)], dtype=bool)
                for tau in range(1, V + 1):
                    v = O.sample_set(keys, nuc, tau)
                    for c in range(V):
                        assert O.in_set_by_rank_count(keys, nuc, tau, c) == (c in v)
    # random at the real vocabulary sizes
    for V in (1025, 2049):
        l32 = (g.standard_normal(V) * 0.64).astype(np.float32)
        keys = O.decision_keys(l32, 1.0, 9, 1, 77)
        nuc = O.nucleus_sorted(l32, 1.0, 0.9)
        for tau in (1, 3, 5):
            v = O.sample_set(keys, nuc, tau)
            assert len(v) == tau and len(set(v)) == tau
            for c in list(g.integers(0, V, 50)) + v:
                assert O.in_set_by_rank_count(keys, nuc, tau, int(c)) == (int(c) in v)


def test_draw_sets_are_nested_in_tau():
    g = np.random.default_rng(6)
    l32 = g.standard_normal(100).astype(np.float32)
    keys = O.decision_keys(l32, 1.0, 1, 0, 0)
    nuc = O.nucleus_sorted(l32, 1.0, 0.95)
    prev = []
    for tau in range(1, 8):
        v = O.sample_set(keys, nuc, tau)
        assert v[:len(prev)] == prev
        prev = v


def test_topk_order_and_ties():
    l = np.array([1.0, 3.0, 3.0, -2.0, 0.5], dtype=np.float32)
    assert list(O.topk_ids(l, 4)) == [1, 2, 0, 4]
