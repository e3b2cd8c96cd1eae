"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Integers (tokens, accepted lengths, paths, KV slots,
edge bits) must match bit for bit wherever the oracle's decision margin exceeds
1e-3; logits and attention outputs within 1e-4 (fp32 models) / 2e-2 (bf16)."""
import numpy as np
import pytest

import oracle as O
import workloads as W
from harness import (MARGIN, MARGINS, TOL, assert_floors, expected_slots, inject_kv, lockstep, make_gpu, read_kv,
                     read_kv_rows, tokens_with_phonemes)

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def _sampling(wl, seed=7, tau=None, temperature=None, top_p=1.0, accept_rule=0):
    import paper_2410_21951_b200 as P
    tau = wl.tau if tau is None else tau
    t = wl.temperature if temperature is None else temperature
    return (O.Sampling(tau=tau, temperature=t, top_p=top_p, seed=seed, accept_rule=accept_rule),
            P.Sampling.make(tau=tau, temperature=t, top_p=top_p, seed=seed, accept_rule=accept_rule))


def _prefill_both(wl, g, table, model, seqs, oracle_chunk=128):
    """GPU prefill of every sequence of the workload; oracle prefill of `seqs`."""
    prefixes = [W.prefix_for(wl, b) for b in range(wl.batch)]
    toks = [tokens_with_phonemes(wl.shape, ph, pr) for ph, pr in prefixes]
    stride = max(len(t) for t in toks)
    mat = np.zeros((wl.batch, stride), dtype=np.int32)
    for b, t in enumerate(toks):
        mat[b, :len(t)] = t
    g.begin(table)
    g.prefill(mat, [len(t) for t in toks])
    states = {b: O.prefill_blocked(model, prefixes[b][0], prefixes[b][1], seq=b, chunk=oracle_chunk) for b in seqs}
    lens = g.lengths()
    for b, st in states.items():
        assert lens[b] == st.S == len(toks[b])
    return states, toks


def _setup(wl, n_iters, seqs, seed=11, extra=0):
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    need = []
    for b in range(wl.batch):
        ph, pr = W.prefix_for(wl, b)
        need.append(len(ph) + len(pr) + n_iters * (tpl.max_depth + 1) + wl.tree_nodes + extra)
    g, table = make_gpu(wl.shape, w, wl.batch, wl.tree_nodes, need, seed)
    g.set_tree(tpl.parent, tpl.rank)
    return w, model, tpl, g, table


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_toy_lockstep_prefill_and_kv(dtype):
    """Small model, several tiles worth of context after prefill, ragged prefix; also
    checks that the committed K/V rows equal the oracle's."""
    wl = W.toy_workload(dtype=dtype, d_model=128, n_heads=2, d_ffn=256, vocab=203, tree_nodes=16, tree_caps=(6, 3, 2),
                        tau=3, temperature=1.0, batch=3, phoneme_len=(20, 70), prompt_len=90, index=11)
    w, model, tpl, g, table = _setup(wl, 6, range(3))
    states, _ = _prefill_both(wl, g, table, model, range(3), oracle_chunk=37)
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 6, dtype, oracle_mode="memo", check_attn=True)
    assert rep.accept_checked > 0 and rep.root_checked > 0 and rep.draft_sets_checked > 0
    for b, st in states.items():
        K, V = read_kv(g, table, b, st.S)
        assert np.abs(K - st.kv.K[:, :st.S]).max() <= TOL[dtype]
        assert np.abs(V - st.kv.V[:, :st.S]).max() <= TOL[dtype]
    g.check()


@pytest.mark.parametrize("dtype,rows", [("fp32", 0), ("bf16", 5), ("bf16", 64)])
def test_prefill_in_passes_of_many_chunks_and_behind_existing_context(dtype, rows):
    """The prefix goes in as two calls (the second one behind what the first left in the cache), with
    0 (= one chunk per sequence and pass), 5 and 64 chunks per pass: the K/V rows, lengths and the carried
    state (through the next iteration's root and logits) equal the oracle's."""
    import paper_2410_21951_b200 as P
    wl = W.toy_workload(dtype=dtype, d_model=128, n_heads=2, d_ffn=256, vocab=203, tree_nodes=16, tree_caps=(6, 3, 2),
                        tau=3, temperature=1.0, batch=3, phoneme_len=(20, 70), prompt_len=90, index=15)
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    prefixes = [W.prefix_for(wl, b) for b in range(wl.batch)]
    toks = [tokens_with_phonemes(wl.shape, ph, pr) for ph, pr in prefixes]
    need = [len(t) + 3 * (tpl.max_depth + 1) + wl.tree_nodes for t in toks]
    table, total = W.shuffled_block_table(need, 64, 21, spare_pages=3)
    g = P.Vadusa(wl.shape, w, max_batch=wl.batch, max_tree_nodes=wl.tree_nodes, max_blocks_per_seq=table.shape[1],
                 kv_num_blocks=total, prefill_rows=rows)
    g.set_tree(tpl.parent, tpl.rank)
    g.begin(table)
    cut = [len(t) // 3 + b for b, t in enumerate(toks)]
    for part in (0, 1):
        seg = [t[:c] if part == 0 else t[c:] for t, c in zip(toks, cut)]
        mat = np.zeros((wl.batch, max(len(x) for x in seg)), dtype=np.int32)
        for b, x in enumerate(seg):
            mat[b, :len(x)] = x
        g.prefill(mat, [len(x) for x in seg])
        want = cut if part == 0 else [len(t) for t in toks]
        assert list(g.lengths()) == want
    states = {b: O.prefill_blocked(model, prefixes[b][0], prefixes[b][1], seq=b, chunk=41) for b in range(wl.batch)}
    for b, st in states.items():
        K, V = read_kv(g, table, b, st.S)
        assert np.abs(K - st.kv.K[:, :st.S]).max() <= TOL[dtype]
        assert np.abs(V - st.kv.V[:, :st.S]).max() <= TOL[dtype]
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 3, dtype, oracle_mode="memo")
    assert rep.iterations == 3
    g.check()


def test_prefill_of_4000_tokens_bf16_pairs_of_chunks():
    """The prefilling pass (Fig. 1a) over long prefixes with 64-token chunks, head_dim 64, bf16: attention runs on
    pairs of consecutive chunks (128 query rows per K/V page).  Two sequences of 4000 and 1531 tokens, fed in two
    calls (the first leaves 37 and 64 tokens, so the second call's chunks start at unaligned and at aligned
    positions, and one sequence has an odd number of chunks): every K/V row and the carried state (through the
    first iteration's logits and decisions) against the oracle."""
    import paper_2410_21951_b200 as P
    wl = W.toy_workload(dtype="bf16", d_model=128, n_heads=2, d_ffn=256, vocab=203, tree_nodes=64, tree_caps=(10, 5, 3),
                        tau=3, temperature=1.0, batch=2, phoneme_len=(60, 100), prompt_len=1471, index=23, max_pos=4200)
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    prefixes = [W.prefix_for(wl, b) for b in range(wl.batch)]
    # sequence 0: a longer prompt (4000 tokens in all)
    ph0 = prefixes[0][0]
    prefixes[0] = (ph0, W.markov_prompt(4000 - len(ph0), wl.shape.vocab - 1, wl.seed(50)))
    toks = [tokens_with_phonemes(wl.shape, ph, pr) for ph, pr in prefixes]
    assert len(toks[0]) == 4000
    need = [len(t) + 2 * (tpl.max_depth + 1) + wl.tree_nodes for t in toks]
    table, total = W.shuffled_block_table(need, 64, 29, spare_pages=2)
    g = P.Vadusa(wl.shape, w, max_batch=wl.batch, max_tree_nodes=wl.tree_nodes, max_blocks_per_seq=table.shape[1],
                 kv_num_blocks=total, prefill_rows=64)
    g.set_tree(tpl.parent, tpl.rank)
    g.begin(table)
    cut = [37, 64]
    for part in (0, 1):
        seg = [t[:c] if part == 0 else t[c:] for t, c in zip(toks, cut)]
        mat = np.zeros((wl.batch, max(len(x) for x in seg)), dtype=np.int32)
        for b, x in enumerate(seg):
            mat[b, :len(x)] = x
        g.prefill(mat, [len(x) for x in seg])
    assert list(g.lengths()) == [len(t) for t in toks]
    states = {b: O.prefill_blocked(model, prefixes[b][0], prefixes[b][1], seq=b, chunk=128) for b in range(wl.batch)}
    for b, st in states.items():
        K, V = read_kv(g, table, b, st.S)
        assert np.abs(K - st.kv.K[:, :st.S]).max() <= TOL["bf16"]
        assert np.abs(V - st.kv.V[:, :st.S]).max() <= TOL["bf16"]
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 2, "bf16", oracle_mode="tree", check_attn=True)
    assert rep.iterations == 2 and rep.root_checked >= 3
    g.check()


@pytest.mark.parametrize("nodes", [10, 24, 48])
def test_bf16_small_token_counts_take_the_layernorm_fused_products(nodes):
    """d_model 256 (two groups of 128 features), one sequence: the token count selects the 16-, 32- and
    64-wide tiles of the products that normalise their own operand from the producer's statistics;
    prefill tails exercise short tiles as well."""
    wl = W.toy_workload(dtype="bf16", d_model=256, n_heads=4, d_ffn=512, vocab=203, tree_nodes=nodes,
                        tree_caps=(6, 3, 2), tau=3, temperature=1.0, batch=1, phoneme_len=(13, 13), prompt_len=70,
                        index=14)
    w, model, tpl, g, table = _setup(wl, 5, range(1))
    states, _ = _prefill_both(wl, g, table, model, range(1), oracle_chunk=29)
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 5, "bf16", oracle_mode="memo", check_attn=True)
    assert rep.iterations == 5 and rep.accept_checked + rep.accept_undecidable == 5
    g.check()


@pytest.mark.parametrize("dtype,tau,temperature,top_p,rule", [("fp32", 2, 0.9, 0.8, 0), ("fp32", 3, 1.0, 1.0, 1),
                                                               ("bf16", 5, 0.8, 1.0, 0), ("fp32", 1, 0.0, 1.0, 0)])
def test_toy_planted_paths_are_accepted(dtype, tau, temperature, top_p, rule):
    """The true continuation planted on the leftmost branch: several tokens are committed
    per iteration and K/V rows move; nucleus and plain top-tau rules included."""
    wl = W.toy_workload(dtype=dtype, d_model=64, n_heads=2, d_ffn=128, vocab=61, tree_nodes=12, tree_caps=(4, 3, 2),
                        batch=2, phoneme_len=(9, 9), prompt_len=60, index=12)
    w, model, tpl, g, table = _setup(wl, 8, range(2))
    states, _ = _prefill_both(wl, g, table, model, range(2))
    so, sg = _sampling(wl, seed=3, tau=tau, temperature=temperature, top_p=top_p, accept_rule=rule)
    # truth under tolerance 1 (plain AR with the same noise)
    so1 = O.Sampling(tau=1, temperature=temperature, top_p=top_p, seed=3, accept_rule=rule)
    planted = {}
    for b in range(2):
        ph, pr = W.prefix_for(wl, b)
        planted[b] = O.ar_decode(model, O.prefill(model, ph, pr, seq=b), so1, 40)
    rep = lockstep(g, table, model, states, tpl, so, sg, 8, dtype, oracle_mode="memo", planted=planted)
    if rule == 0:            # under rule 1 the noisy truth need not be among the plain top-tau
        assert max(rep.accept_lens) == tpl.max_depth + 1
    # the kernel's acceptance statistics (input of the sparse-tree construction, Sec. II-D) count the same tests
    tested, accepted = g.accept_stats()
    assert np.array_equal(tested, rep.tested) and np.array_equal(accepted, rep.accepted)
    assert tested.sum() > 0 and (rule != 0 or accepted[1:].sum() > 0)
    if tau == 1:
        for b, st in states.items():
            assert st.tokens == planted[b][:len(st.tokens)]
    g.check()


def test_unmasked_eos_ends_a_sequence_and_drops_what_follows_it():
    """EOS not masked: (1) EOS planted in the middle of a forced path: the path is cut behind it, the
    sequence becomes inactive and later iterations leave it alone; (2) free-running generation of a
    9-token vocabulary stops where the oracle's does, on seeds whose decisions are all decidable."""
    import torch
    import paper_2410_21951_b200 as P
    wl = W.toy_workload(dtype="fp32", d_model=64, n_heads=2, d_ffn=128, vocab=9, tree_nodes=14, tree_caps=(3, 2, 2),
                        batch=2, phoneme_len=(9, 9), prompt_len=40, index=17, gen_tokens=40)
    w, model, tpl, g, table = _setup(wl, 45, range(2))
    eos = wl.shape.vocab - 1
    dev = g.dev
    # (1) planted
    states, _ = _prefill_both(wl, g, table, model, range(2))
    so = O.Sampling(tau=1, temperature=0.0, eos_masked=False)
    sg = P.Sampling.make(tau=1, temperature=0.0, eos_masked=0)
    rank0 = [n for n in range(tpl.n_nodes) if all(r == 0 for r in tpl.rank_path(n))]
    assert len(rank0) == 4
    g.draft(sg)
    ov = np.tile(np.arange(tpl.n_nodes, dtype=np.int32) % 7, (2, 1))
    ov[0, rank0[1]] = eos                                   # sequence 0: EOS at depth 1 of the forced path
    forced = np.array([rank0[3], rank0[2]], dtype=np.int32)
    acc = torch.zeros(2, dtype=torch.int32, device=dev)
    ptoks = torch.zeros(2, 16, dtype=torch.int32, device=dev)
    g.verify_step(override=torch.from_numpy(ov).to(dev))
    g.accept_and_commit(sg, forced_best=torch.from_numpy(forced).to(dev), accept_len=acc, path_tokens=ptoks)
    for b in range(2):
        tr = O.vadusa_iteration(model, states[b], tpl, so, mode="memo", tokens_override=ov[b], forced_best=int(forced[b]))
        assert int(acc[b]) == tr.accept_len and list(ptoks[b, :tr.accept_len].cpu().numpy()) == tr.path_tokens
    assert int(acc[0]) == 2 and int(acc[1]) == 3 and states[0].finished and not states[1].finished
    lens = g.lengths().copy()
    g.draft(sg); g.verify_step(); g.accept_and_commit(sg, accept_len=acc)
    assert int(acc[0]) == 0 and g.lengths()[0] == lens[0] and g.lengths()[1] > lens[1]
    # (2) free-running
    checked = 0
    for seed in range(8):
        so = O.Sampling(tau=2, temperature=1.0, eos_masked=False, seed=seed)
        sg = P.Sampling.make(tau=2, temperature=1.0, eos_masked=0, seed=seed)
        states, _ = _prefill_both(wl, g, table, model, range(2))
        traces = {b: O.vadusa_generate(model, states[b], tpl, so, 40, mode="memo") for b in range(2)}
        margin = min(min(t.margin_root, t.margin_accept, float(t.margin_draft.min())) for ts in traces.values() for t in ts)
        if margin <= MARGIN:
            continue
        out = torch.full((2, 40), -1, dtype=torch.int32, device=dev)
        out_len = torch.zeros(2, dtype=torch.int32, device=dev)
        g.generate(sg, 40, out, out_len)
        for b in range(2):
            want = states[b].tokens[:40]
            n = int(out_len[b])
            assert n == len(want) and list(out[b, :n].cpu().numpy()) == want
            assert states[b].finished == (eos in want)
        checked += 1
    assert checked >= 2
    g.check()


@pytest.mark.parametrize("dtype,nodes", [("bf16", 96), ("fp32", 128), ("bf16", 128)])
def test_trees_of_96_and_128_nodes(dtype, nodes):
    """The paper's larger candidate trees (Sec. III-A.3): two ancestor words per node, two 64-node query tiles per
    (head, sequence); tensor-core attention (bf16, head_dim 64) and the plain one (fp32); prefill in 96/128-token
    chunks; planted continuation so that deep paths are accepted."""
    wl = W.toy_workload(dtype=dtype, d_model=128, n_heads=2, d_ffn=256, vocab=203, n_draft_heads=4, tree_nodes=nodes,
                        tree_caps=(10, 5, 3, 2), tau=3, temperature=1.0, batch=2, phoneme_len=(20, 60), prompt_len=150,
                        index=18)
    w, model, tpl, g, table = _setup(wl, 4, range(2))
    assert [int((tpl.depth == d).sum()) for d in range(5)] == {96: [1, 9, 30, 42, 14], 128: [1, 10, 35, 53, 29]}[nodes]
    states, _ = _prefill_both(wl, g, table, model, range(2), oracle_chunk=53)
    so, sg = _sampling(wl)
    so1 = O.Sampling(tau=1, temperature=1.0, top_p=1.0, seed=so.seed, accept_rule=0)
    planted = {}
    for b in range(2):
        ph, pr = W.prefix_for(wl, b)
        planted[b] = O.ar_decode(model, O.prefill(model, ph, pr, seq=b), so1, 24)
    rep = lockstep(g, table, model, states, tpl, so, sg, 4, dtype, oracle_mode="memo", check_attn=True, planted=planted)
    assert rep.iterations == 4 and max(rep.accept_lens) == 5
    g.check()


def test_large_vocabulary_of_16001_tokens():
    """The paper's largest codebook (wav2vec 2.0 tokens, top-16000, Sec. III-D): the vocabulary heads, the draft
    top-k and the acceptance test at a 16-times larger vocabulary, nucleus on."""
    wl = W.toy_workload(dtype="bf16", d_model=128, n_heads=2, d_ffn=256, vocab=16001, n_draft_heads=3, tree_nodes=16,
                        tree_caps=(6, 3, 2), tau=4, temperature=0.9, batch=2, phoneme_len=(9, 9), prompt_len=60, index=19)
    w, model, tpl, g, table = _setup(wl, 4, range(2))
    states, _ = _prefill_both(wl, g, table, model, range(2))
    so, sg = _sampling(wl, top_p=0.95)
    rep = lockstep(g, table, model, states, tpl, so, sg, 4, "bf16", oracle_mode="memo")
    assert rep.iterations == 4 and rep.root_checked + rep.draft_sets_checked > 0
    g.check()


def test_logit_bias_hook_follows_the_oracle():
    """The sampler hook: a per-sequence bias on the base head's logits (some tokens banned) in the root sample, the
    tau draws of the acceptance test and the next root; planted continuation decoded under the same bias."""
    import torch
    from dataclasses import replace
    wl = W.toy_workload(dtype="fp32", d_model=64, n_heads=2, d_ffn=128, vocab=61, tree_nodes=12, tree_caps=(4, 3, 2),
                        batch=2, phoneme_len=(9, 9), prompt_len=60, index=22)
    w, model, tpl, g, table = _setup(wl, 8, range(2))
    states, _ = _prefill_both(wl, g, table, model, range(2))
    rng = np.random.Generator(np.random.Philox(key=[22, 1]))
    bias = rng.normal(0, 1.5, size=(2, wl.shape.vocab)).astype(np.float32)
    bias[0, [3, 11, 40]] = -np.inf
    bias[1, [0, 59]] = -np.inf
    so, sg = _sampling(wl, seed=6, tau=2, temperature=0.9, top_p=0.9)
    so = replace(so, bias=bias)
    g.set_logit_bias(torch.from_numpy(bias).to(g.dev))
    so1 = O.Sampling(tau=1, temperature=0.9, top_p=0.9, seed=6, bias=bias)
    planted = {}
    for b in range(2):
        ph, pr = W.prefix_for(wl, b)
        planted[b] = O.ar_decode(model, O.prefill(model, ph, pr, seq=b), so1, 40)
    rep = lockstep(g, table, model, states, tpl, so, sg, 8, "fp32", oracle_mode="memo", planted=planted)
    assert rep.root_checked > 0 and rep.accept_checked > 0 and max(rep.accept_lens) == tpl.max_depth + 1
    for b, banned in ((0, {3, 11, 40}), (1, {0, 59})):
        assert not set(states[b].tokens) & banned
    g.set_logit_bias(None)
    g.check()


def test_degenerate_trees_root_only_and_deepest_chain():
    """A one-node tree is plain decoding (one token per iteration); a chain of 16 nodes over 15 draft heads is the
    deepest path the interface allows: planted, all 16 tokens are committed in one iteration."""
    import torch
    import paper_2410_21951_b200 as P
    # root only
    wl = W.toy_workload(dtype="fp32", d_model=64, n_heads=2, d_ffn=128, vocab=61, n_draft_heads=1, tree_nodes=1,
                        tree_caps=(1,), batch=2, phoneme_len=(5, 9), prompt_len=30, index=20)
    w, model, tpl, g, table = _setup(wl, 12, range(2))
    assert tpl.n_nodes == 1
    states, _ = _prefill_both(wl, g, table, model, range(2))
    so, sg = _sampling(wl, seed=9, tau=2, temperature=0.7)
    rep = lockstep(g, table, model, states, tpl, so, sg, 10, "fp32", oracle_mode="memo")
    assert rep.accept_lens == [1] * 20
    so1 = O.Sampling(tau=1, temperature=0.7, top_p=1.0, seed=9)
    for b in range(2):
        ph, pr = W.prefix_for(wl, b)
        assert states[b].tokens == O.ar_decode(model, O.prefill(model, ph, pr, seq=b), so1, 10)
    g.check()
    g.close()
    # chain of 16 over 15 heads
    wl = W.toy_workload(dtype="bf16", d_model=64, n_heads=2, d_ffn=128, vocab=61, n_draft_heads=15, tree_nodes=16,
                        tree_caps=tuple([1] * 15), batch=1, phoneme_len=(7, 7), prompt_len=40, index=21)
    tpl = W.chain_template(16)
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    need = [sum(len(x) for x in W.prefix_for(wl, 0)) + 3 * 16 + 16]
    g, table = make_gpu(wl.shape, w, 1, 16, need, 13, draft_topk=4)
    g.set_tree(tpl.parent, tpl.rank)
    states, _ = _prefill_both(wl, g, table, model, range(1))
    so, sg = _sampling(wl, seed=4, tau=1, temperature=0.0)
    ph, pr = W.prefix_for(wl, 0)
    planted = {0: O.ar_decode(model, O.prefill(model, ph, pr, seq=0), so, 40)}
    rep = lockstep(g, table, model, states, tpl, so, sg, 2, "bf16", oracle_mode="memo", planted=planted)
    assert max(rep.accept_lens) == 16
    g.check()


def test_six_draft_heads_accept_up_to_seven_tokens():
    """The paper's six-head ablation (Sec. III-A.3): depth-6 tree, planted continuation, paths of 7 tokens."""
    from workloads.trees import _from_rank_paths
    wl = W.toy_workload(dtype="fp32", d_model=64, n_heads=2, d_ffn=128, vocab=61, n_draft_heads=6, tree_nodes=20,
                        tree_caps=(4, 3, 2, 2, 2, 2), batch=2, phoneme_len=(9, 9), prompt_len=60, index=16)
    zero = tuple([0] * 6)
    paths = [zero[:k] for k in range(7)] + [(1,), (2,), (3,), (0, 1), (0, 2), (1, 0), (0, 0, 1), (1, 0, 0), (0, 0, 0, 1),
                                            (0, 0, 0, 0, 1), (0, 0, 0, 0, 0, 1), (0, 1, 0), (0, 1, 0, 0)]
    tpl = _from_rank_paths(paths)
    W.validate_template(tpl, wl.tree_caps)
    assert tpl.n_nodes == 20 and tpl.max_depth == 6
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    need = [sum(len(x) for x in W.prefix_for(wl, b)) + 6 * 7 + wl.tree_nodes for b in range(2)]
    g, table = make_gpu(wl.shape, w, wl.batch, wl.tree_nodes, need, 11)
    g.set_tree(tpl.parent, tpl.rank)
    states, _ = _prefill_both(wl, g, table, model, range(2))
    so, sg = _sampling(wl, seed=5, tau=2, temperature=0.9)
    so1 = O.Sampling(tau=1, temperature=0.9, top_p=1.0, seed=5, accept_rule=0)
    planted = {}
    for b in range(2):
        ph, pr = W.prefix_for(wl, b)
        planted[b] = O.ar_decode(model, O.prefill(model, ph, pr, seq=b), so1, 50)
    rep = lockstep(g, table, model, states, tpl, so, sg, 6, "fp32", oracle_mode="memo", planted=planted)
    assert max(rep.accept_lens) == 7
    g.check()


def test_c1_generate_matches_oracle_and_plain_ar():
    """Configuration 1 (2 layers, d 256, fp32, 16-node tree) end to end: free-running vadusa_generate (greedy,
    tolerance 1, 100 tokens) equals the oracle's speculative decoding and plain AR decoding token for token
    up to the first position where the oracle's top-2 margin is below 1e-3."""
    torch = _torch()
    wl = W.workload("C1")
    w, model, tpl, g, table = _setup(wl, wl.gen_tokens, [0])
    states, toks = _prefill_both(wl, g, table, model, [0])
    so, sg = _sampling(wl)
    ph, pr = W.prefix_for(wl, 0)
    ar_state = O.prefill(model, ph, pr)
    truth, first_thin = [], None
    for i in range(wl.gen_tokens):
        l32 = O.sampling.masked_logits32(ar_state.logits_star, model.eos_id, True)
        top2 = np.sort(l32)[-2:]
        if first_thin is None and top2[1] - top2[0] <= MARGIN:
            first_thin = i
        truth += O.ar_decode(model, ar_state, so, 1)
    out = torch.zeros(1, wl.gen_tokens, dtype=torch.int32, device=g.dev)
    out_len = torch.zeros(1, dtype=torch.int32, device=g.dev)
    stats = g.generate(sg, wl.gen_tokens, out, out_len)
    got = out.cpu().numpy()[0]
    n = wl.gen_tokens if first_thin is None else first_thin
    assert n > 20
    assert list(got[:n]) == truth[:n]
    assert int(out_len.cpu()[0]) == wl.gen_tokens
    assert stats.iterations <= wl.gen_tokens and stats.tokens_generated >= wl.gen_tokens and stats.kernel_launches > 0
    # host-to-host entry gives the same tokens
    mat = toks[0][None, :].copy()
    h_out = np.zeros((1, wl.gen_tokens), dtype=np.int32); h_len = np.zeros(1, dtype=np.int32)
    bt = torch.from_numpy(np.pad(table, ((0, 0), (0, g.cfg.max_blocks_per_seq - table.shape[1])), constant_values=-1)).to(g.dev)
    g.generate_host(sg, bt, mat, np.array([mat.shape[1]], dtype=np.int32), wl.gen_tokens, h_out, h_len)
    assert np.array_equal(h_out[0], got) and h_len[0] == wl.gen_tokens


def test_c1_lockstep_full():
    wl = W.workload("C1")
    w, model, tpl, g, table = _setup(wl, 40, [0])
    states, _ = _prefill_both(wl, g, table, model, [0])
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 40, "fp32", oracle_mode="memo", check_attn=True)
    assert rep.max_logit_err <= 1e-4 and rep.accept_checked >= 35 and rep.attn_checked == 40
    assert_floors(rep, root=0.8, accept=0.85, draft_sets_per_decision=3)
    g.check()


def test_c2_lockstep_64_iterations():
    """Configuration 2 (12 layers, d 1024, 16 heads, bf16, 64-node tree, tolerance 3, temperature 1.0): prefill
    of the 325-token prefix, then 64 iterations in lockstep with the oracle's tree-masked pass, attention
    outputs of every layer included.  Most decisions must be decidable under the bf16 margin."""
    wl = W.workload("C2")
    w, model, tpl, g, table = _setup(wl, 64, [0])
    states, _ = _prefill_both(wl, g, table, model, [0])
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 64, "bf16", oracle_mode="tree", check_attn=True)
    assert rep.iterations == 64 and rep.attn_checked == 64
    assert_floors(rep, root=0.7, accept=0.5, draft_sets_per_decision=2)
    g.check()


def test_c2_free_running_generate_matches_oracle_until_first_undecidable_iteration():
    """Configuration 2, vadusa_generate running on its own (no override, no forced choice): its tokens equal
    the oracle's speculative decoding for as long as every iteration is decidable.  With draft heads accepted at
    chance an iteration commits the root alone; it is decidable when the root sample and every acceptance test
    of the oracle's tree clear the bf16 margin and, in addition, no token that the first draft head could rank
    among its used candidates on the GPU (within the margin of the last used rank) is, or is within the margin
    of being, one of the base head's draws at the root - then the GPU's tree, whatever near-ties it breaks
    differently, accepts nothing either."""
    torch = _torch()
    wl = W.workload("C2")
    n_tok = 28
    w, model, tpl, g, table = _setup(wl, n_tok, [0])
    states, _ = _prefill_both(wl, g, table, model, [0])
    so, sg = _sampling(wl)
    st = states[0]
    used1 = int(tpl.rank[tpl.depth == 1].max()) + 1
    M = MARGINS["bf16"]
    good, iters, stopped = 0, 0, False
    while len(st.tokens) < n_tok:
        l1 = O.sampling.masked_logits32(O.draft_logits(model, st.h_star)[0], model.eos_id, True).astype(np.float64)
        t = O.vadusa_iteration(model, st, tpl, so, mode="tree")
        iters += 1
        if stopped:
            continue
        kth = np.sort(l1)[::-1][used1 - 1]
        maybe = np.nonzero(l1 >= kth - M)[0]
        draws = O.draws_at(model, t.node_logits[0], so, 0, t.S + 1)
        near = any(int(c) in draws or O.decode._edge_margin(model, t.node_logits[0], so, 0, t.S + 1, int(c)) <= M for c in maybe)
        if min(t.margin_root, t.margin_accept) <= M or t.accept_len > 1 or near:
            stopped = True
        else:
            good += 1
    out = torch.full((1, n_tok), -1, dtype=torch.int32, device=g.dev)
    out_len = torch.zeros(1, dtype=torch.int32, device=g.dev)
    g.generate(sg, n_tok, out, out_len)
    got = list(out.cpu().numpy()[0])
    print(f"C2 free-running: {iters} oracle iterations, {good} tokens before the first undecidable iteration")
    assert got[:good] == st.tokens[:good]
    assert good >= 8
    g.check()


def test_c3_batch16_vocab2049_all_sequences():
    """Configuration 3 (batch 16, vocabulary 2049, 42-node tree, tolerance 5, temperature 0.8): the oracle
    follows all 16 sequences for 8 iterations."""
    wl = W.workload("C3")
    seqs = list(range(wl.batch))
    w, model, tpl, g, table = _setup(wl, 8, seqs)
    states, _ = _prefill_both(wl, g, table, model, seqs)
    so, sg = _sampling(wl)
    rep = lockstep(g, table, model, states, tpl, so, sg, 8, "bf16", oracle_mode="tree", check_attn=True)
    assert rep.iterations == 8 and rep.decisions == 128
    assert_floors(rep, root=0.7, accept=0.5, draft_sets_per_decision=2)
    g.check()


def _random_context(model, S, rng, scale=1.0):
    K = O.round_bf16(rng.standard_normal((model.L, S, model.H, model.dh)) * scale)
    V = O.round_bf16(rng.standard_normal((model.L, S, model.H, model.dh)) * scale)
    return K, V


@pytest.mark.parametrize("name", ["C4", "C5"])
def test_long_ragged_contexts_with_injected_kv(name):
    """Configurations 4 (batch 32, contexts 1000-4000, shared 64-node tree) and 5 (batch 64, contexts 256-3000, a
    random topology per sequence) at full batch and context lengths: the KV cache holds seeded random bf16 rows
    (so no prefill is needed on either side), tree tokens and the carried state are random; the oracle scores
    four sampled sequences (shortest, longest, two others).  Configuration 4 goes on with the tolerance sweep
    {1, 3, 5} from the same state (draws of the oracle planted below the root, so that the accepted sets differ
    and grow with the tolerance, Sec. III-B) and with a forced five-token path whose committed K/V rows are read
    back, one of them across a page boundary behind a context of almost 4000 tokens."""
    torch = _torch()
    wl = W.workload(name)
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    B, N = wl.batch, wl.tree_nodes
    lens = W.ragged_lengths(B, wl.context_len[0], wl.context_len[1], wl.seed(900))
    if name == "C4":
        # the longest context ends three rows before a page boundary: a five-token commit crosses it
        lens = lens.copy()
        b_edge = int(np.argmax(lens))
        lens[b_edge] = (int(lens[b_edge]) // 64) * 64 - 3
        assert lens[b_edge] > 3700
    g, table = make_gpu(wl.shape, w, B, N, [int(s) + N + 8 for s in lens], wl.seed(1))
    g.begin(table, ctx_len=lens)
    if wl.random_topology:
        tpls = [W.random_topology(N, wl.topology_max_depth, wl.seed(100 + b)) for b in range(B)]
        g.set_tree(np.stack([t.parent for t in tpls]), np.stack([t.rank for t in tpls]), per_sequence=True)
    else:
        tpls = [W.static_template(N, wl.tree_caps)] * B
        g.set_tree(tpls[0].parent, tpls[0].rank)
    order = np.argsort(lens)
    picks = [int(order[0]), int(order[-1]), int(order[B // 2])]
    # The many-token products run on CTA pairs: each CTA of a pair stages half of a 128- or 256-token
    # tile, i.e. whole sequences of 64 nodes.  One more sequence, so that the samples fall into both
    # halves of both tile widths (b % 4 in {0, 1} and {2, 3}; b even and odd).
    def both_halves(ps):
        return {b % 4 < 2 for b in ps} == {True, False} and {b % 2 for b in ps} == {0, 1}
    picks.append(next(b for b in range(B) if b not in picks and both_halves(picks + [b])))
    if name == "C4" and b_edge not in picks:
        picks.append(b_edge)
    rng = np.random.default_rng(wl.seed(2))
    # every sequence gets random K/V on the GPU; the sampled ones also in the oracle
    view = g.kv_view()
    view.normal_()                                           # all pages: seeded below for the sampled ones
    states = {}
    for b in picks:
        K, V = _random_context(model, int(lens[b]), rng)
        inject_kv(g, table, b, K, V)
        kv = O.KVCache(model, capacity=int(lens[b]) + 80)
        kv.extend(K, V)
        states[b] = kv
    toks = rng.integers(0, wl.shape.vocab - 1, size=(B, N)).astype(np.int32)
    logits = torch.zeros(B, N, wl.shape.vocab, dtype=torch.float32, device=g.dev)
    attn = torch.zeros(model.L, B, N, model.d, dtype=g.tdtype, device=g.dev)
    g.verify_step(override=torch.from_numpy(toks).to(g.dev), logits_out=logits, attn_tap=attn)
    so, sg = _sampling(wl, seed=5)
    acc = torch.zeros(B, dtype=torch.int32, device=g.dev)
    pn = torch.zeros(B, 16, dtype=torch.int32, device=g.dev)
    sl = torch.zeros(B, 16, dtype=torch.int64, device=g.dev)
    eb = torch.zeros(B, dtype=torch.int64, device=g.dev)
    g.accept_and_commit(sg, accept_len=acc, path_nodes=pn, kv_slots=sl, edge_bits=eb)
    lg = logits.cpu().numpy().astype(np.float64)
    at = attn.float().cpu().numpy().astype(np.float64)
    first_pass = {}
    for b in picks:
        tpl = tpls[b]
        mask = np.zeros((N, N), dtype=bool)
        for n in range(N):
            mask[n, tpl.node_path(n)] = True
        S = int(lens[b])
        out = O.forward_tree(model, states[b], [0] * N, toks[b], S + tpl.depth, mask)
        first_pass[b] = out
        e_l = np.abs(lg[b] - out.logits).max()
        e_a = max(np.abs(at[l, b] - out.attn[l]).max() for l in range(model.L))
        print(f"{name} seq {b} (context {int(lens[b])}): max |logit err| {e_l:.2e}, max |attn err| {e_a:.2e}")
        assert e_l <= TOL["bf16"] and e_a <= TOL["bf16"]
        # accept decision of the oracle on its own logits
        draws = {n: O.draws_at(model, out.logits[n], so, b, S + int(tpl.depth[n]) + 1) for n in range(N)}
        ok = O.tree_edge_accepts(tpl.parent, toks[b], draws)
        best, path = O.accept_from_edges(tpl.parent, tpl.depth, ok)
        margin = min(O.decode._edge_margin(model, out.logits[int(tpl.parent[n])], so, b,
                                           S + int(tpl.depth[int(tpl.parent[n])]) + 1, int(toks[b, n]))
                     for n in range(1, N))
        if margin > MARGINS["bf16"]:
            assert int(acc[b]) == len(path) and list(pn[b, :len(path)].cpu().numpy()) == path
            assert list(sl[b, :len(path)].cpu().numpy()) == expected_slots(table, b, S, len(path))
    assert np.array_equal(g.lengths(), lens + acc.cpu().numpy())
    g.check()
    # the same pass through the page-stream attention kernel (opt-in) at the full batch and context lengths
    g.set_attention_stream(True)
    g.begin(table, ctx_len=lens)
    if wl.random_topology:
        g.set_tree(np.stack([t.parent for t in tpls]), np.stack([t.rank for t in tpls]), per_sequence=True)
    g.verify_step(override=torch.from_numpy(toks).to(g.dev), logits_out=logits, attn_tap=attn)
    g.check()
    g.set_attention_stream(False)
    lg2 = logits.cpu().numpy().astype(np.float64)
    at2 = attn.float().cpu().numpy().astype(np.float64)
    for b in picks:
        out = first_pass[b]
        e_l = np.abs(lg2[b] - out.logits).max()
        e_a = max(np.abs(at2[l, b] - out.attn[l]).max() for l in range(model.L))
        print(f"{name} seq {b}, page-stream attention: max |logit err| {e_l:.2e}, max |attn err| {e_a:.2e}")
        assert e_l <= TOL["bf16"] and e_a <= TOL["bf16"]
    if name != "C4":
        return
    # ---- tolerance sweep from the same state: the 1st, 3rd and 5th draw of the oracle at the root planted as
    # the first three candidates below it
    tpl = tpls[0]
    d1 = [n for n in range(N) if tpl.depth[n] == 1]
    toks2 = toks.copy()
    outs = {}
    for b in picks:
        S = int(lens[b])
        mask = np.zeros((N, N), dtype=bool)
        for n in range(N):
            mask[n, tpl.node_path(n)] = True
        root_logits = O.forward_tree(model, states[b], [0] * N, toks[b], S + tpl.depth, mask).logits[0]
        d5 = O.draws_at(model, root_logits, O.Sampling(tau=5, temperature=so.temperature, seed=so.seed), b, S + 1)
        assert len(d5) == 5
        toks2[b, d1[0]], toks2[b, d1[1]], toks2[b, d1[2]] = d5[0], d5[2], d5[4]
        outs[b] = O.forward_tree(model, states[b], [0] * N, toks2[b], S + tpl.depth, mask)
    dev_toks2 = torch.from_numpy(toks2).to(g.dev)
    got = {}
    checked = 0
    for tau in (1, 3, 5):
        so_t, sg_t = _sampling(wl, seed=5, tau=tau)
        g.begin(table, ctx_len=lens)
        g.verify_step(override=dev_toks2)
        g.accept_and_commit(sg_t, accept_len=acc, path_nodes=pn, edge_bits=eb)
        got[tau] = (acc.cpu().numpy().copy(), eb.cpu().numpy().astype(np.uint64).copy())
        for b in picks:
            S, out = int(lens[b]), outs[b]
            draws = {n: O.draws_at(model, out.logits[n], so_t, b, S + int(tpl.depth[n]) + 1) for n in range(N)}
            ok = O.tree_edge_accepts(tpl.parent, toks2[b], draws)
            best, path = O.accept_from_edges(tpl.parent, tpl.depth, ok)
            accd = {0}
            want_bits = 1
            margin = float("inf")
            for n in range(1, N):
                p = int(tpl.parent[n])
                if p in accd:
                    margin = min(margin, O.decode._edge_margin(model, out.logits[p], so_t, b, S + int(tpl.depth[p]) + 1, int(toks2[b, n])))
                    if ok[n]:
                        accd.add(n); want_bits |= 1 << n
            if margin > MARGINS["bf16"]:
                assert int(got[tau][0][b]) == len(path) and list(pn[b, :len(path)].cpu().numpy()) == path
                assert int(got[tau][1][b]) == want_bits, f"tau {tau} seq {b}: {int(got[tau][1][b]):x} != {want_bits:x}"
                assert len(path) >= 2 and (want_bits >> d1[0]) & 1            # the first draw is accepted at any tolerance
                checked += 1
    print(f"C4 tolerance sweep: {checked} of {3 * len(picks)} decisions decidable")
    assert checked >= 6
    # a larger tolerance accepts a superset of edges below the same accepted nodes and never a shorter path
    for lo, hi in ((1, 3), (3, 5)):
        assert np.all(got[lo][0] <= got[hi][0])
        assert np.all((got[lo][1] & ~got[hi][1]) == 0)
    for b in picks:
        assert bin(int(got[5][1][b])).count("1") > bin(int(got[1][1][b])).count("1")
    # ---- a forced five-token path: the committed rows, read back behind up to 3965 context tokens
    leaf = int(np.nonzero(tpl.depth == tpl.max_depth)[0][0])
    path = tpl.node_path(leaf)
    g.begin(table, ctx_len=lens)
    g.verify_step(override=dev_toks2)
    forced = torch.full((B,), leaf, dtype=torch.int32, device=g.dev)
    g.accept_and_commit(sg, forced_best=forced, accept_len=acc, path_nodes=pn, kv_slots=sl)
    assert np.all(acc.cpu().numpy() == len(path))
    crossed = 0
    for b in picks:
        S = int(lens[b])
        assert list(pn[b, :len(path)].cpu().numpy()) == path
        assert list(sl[b, :len(path)].cpu().numpy()) == expected_slots(table, b, S, len(path))
        K, V = read_kv_rows(g, table, b, range(S, S + len(path)))
        assert np.abs(K - outs[b].K[:, path]).max() <= TOL["bf16"] and np.abs(V - outs[b].V[:, path]).max() <= TOL["bf16"]
        crossed += int(S // 64 != (S + len(path) - 1) // 64)
    assert crossed >= 1
    assert np.array_equal(g.lengths(), lens + len(path))
    g.check()


def test_capacity_error_is_reported_not_faulted():
    """A block table too short for context + tree: the device flags it, no access goes out
    of bounds, and the next synchronising call returns ECAPACITY."""
    import paper_2410_21951_b200 as P
    torch = _torch()
    wl = W.toy_workload(dtype="fp32", d_model=64, n_heads=2, d_ffn=128, vocab=61, tree_nodes=12, tree_caps=(4, 3, 2))
    w = W.make_weights(wl.shape, wl.seed())
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    g, table = make_gpu(wl.shape, w, 1, wl.tree_nodes, [64], 1, spare_pages=0)      # one block only
    g.set_tree(tpl.parent, tpl.rank)
    g.begin(table, ctx_len=[60])                                                     # 60 + 12 nodes > 64
    toks = torch.zeros(1, wl.tree_nodes, dtype=torch.int32, device=g.dev)
    g.verify_step(override=toks)
    with pytest.raises(P.VadusaError) as e:
        g.check()
    assert e.value.status == 4


def test_call_order_and_argument_errors():
    import paper_2410_21951_b200 as P
    torch = _torch()
    wl = W.toy_workload(dtype="fp32", d_model=64, n_heads=2, d_ffn=128, vocab=61, tree_nodes=12, tree_caps=(4, 3, 2))
    w = W.make_weights(wl.shape, wl.seed())
    g, table = make_gpu(wl.shape, w, 2, wl.tree_nodes, [200, 200], 1)
    sp = P.Sampling.make(tau=1)
    with pytest.raises(P.VadusaError) as e:
        g.verify_step()
    assert e.value.status == 5                              # no batch begun
    g.begin(table)
    with pytest.raises(P.VadusaError) as e:
        g.draft(sp)
    assert e.value.status == 5                              # no tree
    bad_parent = np.array([-1, 0, 0, 5], dtype=np.int32)    # node 3's parent does not precede it
    with pytest.raises(P.VadusaError) as e:
        g.set_tree(bad_parent, np.zeros(4, dtype=np.int32))
    assert e.value.status == 1
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    with pytest.raises(P.VadusaError):                      # siblings out of rank order
        g.set_tree(tpl.parent, tpl.rank[::-1].copy())
    g.set_tree(tpl.parent, tpl.rank)
    with pytest.raises(P.VadusaError) as e:
        g.verify_step()
    assert e.value.status == 5                              # no draft, no override
    with pytest.raises(P.VadusaError) as e:
        g.accept_and_commit(sp)
    assert e.value.status == 5
    with pytest.raises(P.VadusaError) as e:
        g.draft(P.Sampling.make(tau=0))
    assert e.value.status == 1
