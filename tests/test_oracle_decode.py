"""Pins of the oracle's decoding loop against what the paper fixes: tolerance 1
is plain AR decoding, the worked example of Sec. II-A, Algorithm 1 by brute
force, longest-then-leftmost, nesting in tau, and the state of the cache."""
import itertools
import json
import os

import numpy as np
import pytest

import oracle as O
import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _setup(dtype="fp32", **kw):
    wl = W.toy_workload(dtype=dtype, **kw)
    w = W.make_weights(wl.shape, wl.seed())
    m = O.Model.from_shape(wl.shape, w)
    ph, pr = W.prefix_for(wl, 0)
    return wl, m, ph, pr


def test_worked_example_from_the_paper():
    ex = json.load(open(os.path.join(GOLDEN, "worked_example.json")))
    k_star = O.verify_branch(ex["branch"], ex["draw_sets"])
    assert k_star == ex["expected_k_star"] and k_star + 1 == ex["expected_accept_len"]
    # the same situation through the whole loop: plant the true continuation at
    # depth 1, a wrong token at depth 2, and check what is committed
    wl, m, ph, pr = _setup()
    sp = O.Sampling(tau=1, temperature=0.0)
    truth = O.ar_decode(m, O.prefill(m, ph, pr), sp, 4)
    tpl = W.chain_template(3)
    st = O.prefill(m, ph, pr)
    wrong = (truth[2] + 1) % (wl.shape.vocab - 1)
    tr = O.vadusa_iteration(m, st, tpl, sp, tokens_override=np.array([truth[0], truth[1], wrong]))
    assert tr.accept_len == 2 and tr.path_tokens == truth[:2] and tr.best_node == ex["next_root_comes_from_node"]
    # decoding continues from the base head's prediction at the last accepted token
    assert O.sample_next(m, st.logits_star, sp, 0, st.S) == truth[2]


@pytest.mark.parametrize("temperature,top_p", [(0.0, 1.0), (1.0, 1.0), (0.8, 0.9)])
@pytest.mark.parametrize("shape", ["static", "chain", "random"])
def test_tolerance_one_equals_plain_ar(temperature, top_p, shape):
    """Sec. II-A: with a single 'correct token' per position speculative decoding
    is lossless, whatever tree is used."""
    wl, m, ph, pr = _setup()
    tpl = {"static": W.static_template(10, (4, 3, 2)), "chain": W.chain_template(4),
           "random": W.random_topology(12, 3, 123)}[shape]
    sp = O.Sampling(tau=1, temperature=temperature, top_p=top_p, seed=42)
    want = O.ar_decode(m, O.prefill(m, ph, pr), sp, 24)
    st = O.prefill(m, ph, pr)
    traces = O.vadusa_generate(m, st, tpl, sp, 24)
    assert st.tokens[:24] == want
    assert all(1 <= t.accept_len <= tpl.max_depth + 1 for t in traces)


def test_unmasked_eos_ends_the_sequence_exactly_where_plain_ar_ends_it():
    """With EOS unmasked and tolerance 1 the speculative loop still equals plain decoding (Sec. II-A),
    including where it stops; tokens that follow EOS on an accepted path are not committed."""
    wl, m, ph, pr = _setup(vocab=9)                 # 8 speech ids + EOS: EOS turns up within a few tokens
    tpl = W.static_template(10, (4, 3, 2))
    stopped = 0
    for seed in range(6):
        sp = O.Sampling(tau=1, temperature=1.0, eos_masked=False, seed=seed)
        st_ar = O.prefill(m, ph, pr)
        want = O.ar_decode(m, st_ar, sp, 40)
        st = O.prefill(m, ph, pr)
        traces = O.vadusa_generate(m, st, tpl, sp, 40)
        assert st.tokens[:len(want)] == want and st.finished == st_ar.finished
        if st_ar.finished:
            stopped += 1
            assert want[-1] == m.eos_id and m.eos_id not in want[:-1]
            assert st.tokens == want and traces[-1].finished and traces[-1].path_tokens[-1] == m.eos_id
    assert stopped >= 3
    # EOS planted in the middle of a fully accepted path: the rest of the path is dropped
    sp = O.Sampling(tau=1, temperature=0.0, eos_masked=False)
    st = O.prefill(m, ph, pr)
    chain = W.chain_template(4)
    toks = np.array([3, m.eos_id, 5, 6])
    tr = O.vadusa_iteration(m, st, chain, sp, tokens_override=toks, forced_best=3)
    assert tr.finished and tr.accept_len == 2 and tr.path_tokens == [3, m.eos_id] and tr.best_node == 1
    assert st.finished and st.tokens[-2:] == [3, m.eos_id]


def test_logit_bias_reshapes_the_base_head_only_where_it_samples():
    """Sec. II-C, last paragraph: another sampling strategy enters as the original head's predictions.  A zero
    bias changes nothing; banned tokens (-inf) never appear; a dominant bias forces its token; tolerance 1
    stays plain decoding under the same bias."""
    wl, m, ph, pr = _setup()
    V = wl.shape.vocab
    tpl = W.static_template(10, (4, 3, 2))
    base = O.Sampling(tau=2, temperature=1.0, seed=5)
    st0 = O.prefill(m, ph, pr); O.vadusa_generate(m, st0, tpl, base, 16)
    zero = O.Sampling(tau=2, temperature=1.0, seed=5, bias=np.zeros((1, V), dtype=np.float32))
    st1 = O.prefill(m, ph, pr); O.vadusa_generate(m, st1, tpl, zero, 16)
    assert st1.tokens == st0.tokens
    banned = sorted(set(st0.tokens[:6]))
    b = np.zeros((1, V), dtype=np.float32); b[0, banned] = -np.inf
    ban = O.Sampling(tau=2, temperature=1.0, seed=5, bias=b)
    st2 = O.prefill(m, ph, pr); O.vadusa_generate(m, st2, tpl, ban, 16)
    assert not set(st2.tokens) & set(banned)
    b = np.zeros((1, V), dtype=np.float32); b[0, 7] = 1e4
    st3 = O.prefill(m, ph, pr); O.vadusa_generate(m, st3, tpl, O.Sampling(tau=1, temperature=0.9, seed=1, bias=b), 8)
    assert set(st3.tokens) == {7}
    g = np.random.Generator(np.random.Philox(key=[3, 3]))
    b = g.normal(0, 2.0, size=(1, V)).astype(np.float32)
    sp1 = O.Sampling(tau=1, temperature=1.0, seed=9, bias=b)
    want = O.ar_decode(m, O.prefill(m, ph, pr), sp1, 20)
    st4 = O.prefill(m, ph, pr); O.vadusa_generate(m, st4, tpl, sp1, 20)
    assert st4.tokens[:20] == want
    assert want != O.ar_decode(m, O.prefill(m, ph, pr), O.Sampling(tau=1, temperature=1.0, seed=9), 20)


def test_planted_continuation_is_fully_accepted_and_cache_equals_ar_cache():
    """If the tree holds the true continuation, all of it is accepted (tau = 1),
    and afterwards the cache holds exactly what plain AR decoding stores."""
    wl, m, ph, pr = _setup()
    sp = O.Sampling(tau=1, temperature=1.0, seed=3)
    ar = O.prefill(m, ph, pr)
    truth = O.ar_decode(m, ar, sp, 9)
    tpl = W.static_template(10, (4, 3, 2))
    st = O.prefill(m, ph, pr)
    total = 0
    for it in range(3):
        S0 = st.S
        base = O.vadusa_iteration(m, O.prefill(m, ph, pr) if it == 0 else _clone(m, st), tpl, sp)
        toks = base.tree_tokens.copy()
        # plant truth along the path of ranks (1, 0, 1): nodes found by rank path
        want_path = [n for n in range(tpl.n_nodes) if tpl.rank_path(n) in [(), (1,), (1, 0), (1, 0, 1)]]
        for j, n in enumerate(want_path):
            toks[n] = truth[total + j]
        tr = O.vadusa_iteration(m, st, tpl, sp, tokens_override=toks)
        assert tr.accept_len == len(want_path) and tr.path_nodes == want_path
        total += tr.accept_len
        assert st.S == S0 + tr.accept_len
    n = st.S
    assert st.tokens == truth[:total]
    ar2 = O.prefill(m, ph, pr); O.ar_decode(m, ar2, sp, total)
    assert np.array_equal(st.kv.K[:, :n], ar2.kv.K[:, :n]) and np.array_equal(st.kv.V[:, :n], ar2.kv.V[:, :n])
    assert np.array_equal(st.logits_star, ar2.logits_star)


def _clone(m, st):
    kv = O.KVCache(m, capacity=st.kv.K.shape[1])
    kv.extend(st.kv.K[:, :st.kv.n].copy(), st.kv.V[:, :st.kv.n].copy())
    return O.State(kv=kv, tokens=list(st.tokens), h_star=st.h_star.copy(), logits_star=st.logits_star.copy(), seq=st.seq)


def test_modes_agree():
    wl, m, ph, pr = _setup()
    tpl = W.static_template(10, (4, 3, 2))
    sp = O.Sampling(tau=3, temperature=1.0, seed=8)
    a, b, c = (O.prefill(m, ph, pr) for _ in range(3))
    for _ in range(4):
        ta = O.vadusa_iteration(m, a, tpl, sp, mode="branch")
        tb = O.vadusa_iteration(m, b, tpl, sp, mode="memo")
        tc = O.vadusa_iteration(m, c, tpl, sp, mode="tree")
        assert np.array_equal(ta.node_logits, tb.node_logits)
        assert np.allclose(ta.node_logits, tc.node_logits, atol=1e-10)
        assert ta.path_nodes == tb.path_nodes == tc.path_nodes
        assert ta.path_tokens == tb.path_tokens == tc.path_tokens


def test_algorithm1_brute_force_on_small_trees():
    """Every pattern of accepted edges on small trees: per-branch Algorithm 1 plus
    longest-then-leftmost equals the whole-tree form."""
    shapes = [W.static_template(n, caps) for n, caps in [(5, (3, 2)), (8, (3, 2, 2)), (10, (4, 3, 2))]]
    shapes += [W.random_topology(9, 4, s) for s in range(4)] + [W.chain_template(5)]
    for tpl in shapes:
        N = tpl.n_nodes
        leaves = tpl.leaves()
        toks = np.arange(100, 100 + N)                       # distinct tokens
        for bits in range(2 ** (N - 1)):
            edge = np.array([True] + [(bits >> (n - 1)) & 1 == 1 for n in range(1, N)])
            sets = {p: [int(toks[c]) for c in tpl.children(p) if edge[c]] for p in range(N)}
            res = []
            for leaf in leaves:
                path = tpl.node_path(leaf)
                k_star = O.verify_branch([int(toks[n]) for n in path], [sets[n] for n in path[:-1]] + [[]])
                res.append((tpl.rank_path(leaf), k_star))
            win = O.select_best(res)
            want_path = tpl.node_path(leaves[win])[: res[win][1] + 1]
            ok = O.tree_edge_accepts(tpl.parent, toks, sets)
            assert np.array_equal(ok, edge)
            best, path = O.accept_from_edges(tpl.parent, tpl.depth, ok)
            assert path == want_path and best == want_path[-1]
            # brute-force statement of the rule itself
            accepted = [n for n in range(N) if all(edge[a] for a in tpl.node_path(n))]
            deepest = max(tpl.depth[n] for n in accepted)
            assert best == min((n for n in accepted if tpl.depth[n] == deepest), key=lambda n: tpl.rank_path(n))


def test_longest_then_leftmost():
    assert O.select_best([((0, 0), 1), ((1, 0), 2), ((2, 1), 2)]) == 1      # longest wins, then leftmost
    assert O.select_best([((3,), 0), ((0, 1), 0)]) == 0                      # nothing accepted: root only
    assert O.select_best([((1, 0, 0), 1), ((0, 2, 0), 1)]) == 1              # equal length: smaller ranks


def test_accept_length_is_monotone_in_tau():
    """A larger tolerance can only add 'correct tokens' (the draw sets are nested),
    so from one state the accepted length cannot shrink (paper, ablation on tau)."""
    wl, m, ph, pr = _setup(vocab=21)
    tpl = W.static_template(10, (4, 3, 2))
    st = O.prefill(m, ph, pr)
    grew = 0
    for it in range(6):
        lens = []
        for tau in (1, 2, 3, 5, 20):
            sp = O.Sampling(tau=tau, temperature=1.0, seed=it)
            lens.append(O.vadusa_iteration(m, _clone(m, st), tpl, sp, mode="memo").accept_len)
        assert lens == sorted(lens)
        grew += lens[-1] > lens[0]
        # tau = number of non-EOS tokens: every candidate is a draw, so a deepest leaf wins
        assert lens[-1] == tpl.max_depth + 1
        O.vadusa_iteration(m, st, tpl, O.Sampling(tau=1, temperature=1.0, seed=it), mode="memo")
    assert grew > 0


def test_accept_rule_plain_topk_ignores_noise_for_membership():
    wl, m, ph, pr = _setup()
    tpl = W.static_template(10, (4, 3, 2))
    st = O.prefill(m, ph, pr)
    sp = O.Sampling(tau=3, temperature=1.0, seed=5, accept_rule=1)
    tr = O.vadusa_iteration(m, _clone(m, st), tpl, sp)
    for n in range(1, tpl.n_nodes):
        p = int(tpl.parent[n])
        l = tr.node_logits[p].copy(); l[m.eos_id] = -np.inf
        top3 = sorted(range(m.V), key=lambda j: (-np.float32(l[j]), j))[:3]
        assert tr.edge_ok[n] == (int(tr.tree_tokens[n]) in top3)


def test_full_config_c1_speculative_equals_ar():
    """Configuration 1 (2 layers, d 256, 16-node tree, greedy, tolerance 1, 100 tokens)."""
    wl = W.workload("C1")
    m = O.Model.from_shape(wl.shape, W.make_weights(wl.shape, wl.seed()))
    ph, pr = W.prefix_for(wl, 0)
    sp = O.Sampling(tau=wl.tau, temperature=wl.temperature)
    want = O.ar_decode(m, O.prefill(m, ph, pr), sp, wl.gen_tokens)
    st = O.prefill(m, ph, pr)
    O.vadusa_generate(m, st, W.static_template(wl.tree_nodes, wl.tree_caps), sp, wl.gen_tokens, mode="memo")
    assert st.tokens[:wl.gen_tokens] == want
