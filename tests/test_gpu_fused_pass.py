"""GPU parity of the single-sequence verify pass that runs as one persistent kernel (bf16, head_dim 64,
8 or 16 heads, at most 64 tree nodes): the same lockstep protocol against the CPU oracle as the other
parity tests, on models small enough for the oracle but wide enough for that kernel, plus long contexts
with injected K/V (several groups of pages per CTA, a ragged last page) and a comparison with the
kernel-per-step path on the same state."""
import numpy as np
import pytest

import oracle as O
import workloads as W
from harness import TOL, inject_kv, lockstep, make_gpu, read_kv, tokens_with_phonemes

pytestmark = pytest.mark.gpu


def _wide_toy(nodes, heads=8, d_ffn=2048, vocab=203, layers=2, index=31, phoneme_len=(20, 20), prompt_len=90,
              tree_caps=(6, 3, 2), n_draft_heads=3, max_pos=4096):
    return W.toy_workload(dtype="bf16", n_layers=layers, d_model=64 * heads, n_heads=heads, d_ffn=d_ffn, vocab=vocab,
                          n_draft_heads=n_draft_heads, tree_nodes=nodes, tree_caps=tree_caps, tau=3, temperature=1.0,
                          batch=1, phoneme_len=phoneme_len, prompt_len=prompt_len, index=index, max_pos=max_pos)


def _sampling(wl, seed=7):
    import paper_2410_21951_b200 as P
    return (O.Sampling(tau=wl.tau, temperature=wl.temperature, seed=seed),
            P.Sampling.make(tau=wl.tau, temperature=wl.temperature, seed=seed))


def _start(wl, n_iters, seed=11, prefill_rows=16, cluster=1):
    import paper_2410_21951_b200 as P
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    ph, pr = W.prefix_for(wl, 0)
    toks = tokens_with_phonemes(wl.shape, ph, pr)
    need = [len(toks) + n_iters * (tpl.max_depth + 1) + wl.tree_nodes + 8]
    table, total = W.shuffled_block_table(need, 64, seed, spare_pages=3)
    g = P.Vadusa(wl.shape, w, max_batch=1, max_tree_nodes=wl.tree_nodes, max_blocks_per_seq=table.shape[1],
                 kv_num_blocks=total, prefill_rows=prefill_rows)
    g.set_fused_pass(cluster)
    g.set_tree(tpl.parent, tpl.rank)
    g.begin(table)
    g.prefill(toks[None, :].copy(), [len(toks)])
    st = O.prefill_blocked(model, ph, pr, seq=0, chunk=47)
    assert g.lengths()[0] == st.S
    return w, model, tpl, g, table, st, (ph, pr)


@pytest.mark.parametrize("heads,nodes,rows,cluster", [(8, 16, 16, 8), (8, 48, 0, 6), (16, 64, 0, 1), (16, 37, 16, 6)])
def test_fused_pass_lockstep_against_the_oracle(heads, nodes, rows, cluster):
    """Lockstep iterations (logits, attention outputs per layer, draft, acceptance, committed K/V rows).  With
    prefill_rows = 0 the prefix chunks also go through the persistent kernel, one chunk per pass.  Clusters of
    8 CTAs (K slices of equal width, 8 tokens per owner) and of 6 (uneven K slices and token shares)."""
    caps = (6, 3, 2) if nodes < 64 else (10, 5, 3)
    wl = _wide_toy(nodes, heads=heads, d_ffn=256 * heads, tree_caps=caps, index=31 + heads)
    w, model, tpl, g, table, st, _ = _start(wl, 6, prefill_rows=rows, cluster=cluster)
    so, sg = _sampling(wl)
    launches0 = g.kernel_launches()
    rep = lockstep(g, table, model, {0: st}, tpl, so, sg, 5, "bf16", oracle_mode="memo", check_attn=True)
    assert rep.iterations == 5 and rep.attn_checked == 5
    assert rep.root_checked + rep.draft_sets_checked > 0 and rep.accept_checked + rep.accept_undecidable == 5
    # one launch for the pass: draft (3) + tree tokens (1) + pass (1) + accept, commit (2) per iteration
    assert g.fused_pass_clusters() >= heads, "this device cannot hold one cluster per head"
    assert g.kernel_launches() - launches0 <= 5 * 8
    K, V = read_kv(g, table, 0, st.S)
    assert np.abs(K - st.kv.K[:, :st.S]).max() <= TOL["bf16"]
    assert np.abs(V - st.kv.V[:, :st.S]).max() <= TOL["bf16"]
    g.check()


def test_fused_pass_planted_path_moves_rows_and_matches_stepwise_path():
    """The oracle's plain continuation planted on the leftmost branch (several tokens committed per
    iteration), then the same tree scored by both paths from the same state: the logits of the two paths
    agree far inside the tolerance against the oracle."""
    import torch
    wl = _wide_toy(24, heads=8, index=37)
    w, model, tpl, g, table, st, (ph, pr) = _start(wl, 8)
    so, sg = _sampling(wl, seed=3)
    so1 = O.Sampling(tau=1, temperature=so.temperature, seed=3)
    planted = {0: O.ar_decode(model, O.prefill(model, ph, pr, seq=0), so1, 30)}
    rep = lockstep(g, table, model, {0: st}, tpl, so, sg, 5, "bf16", oracle_mode="memo", check_attn=True, planted=planted)
    assert max(rep.accept_lens) == tpl.max_depth + 1
    N, V = tpl.n_nodes, wl.shape.vocab
    rng = np.random.default_rng(5)
    toks = torch.from_numpy(rng.integers(0, V - 1, size=(1, N)).astype(np.int32)).to(g.dev)
    a = torch.zeros(1, N, V, dtype=torch.float32, device=g.dev)
    b = torch.zeros_like(a)
    g.verify_step(override=toks, logits_out=a)
    g.set_fused_pass(False)
    g.verify_step(override=toks, logits_out=b)
    g.set_fused_pass(True)
    assert float((a - b).abs().max()) <= 1e-2
    g.check()


@pytest.mark.parametrize("ctx_len,cluster", [(37, 8), (1990, 8), (2500, 8), (2500, 6), (700, 0), (1500, 0), (2500, 0)])
def test_fused_pass_long_context_with_injected_kv(ctx_len, cluster):
    """Seeded random K/V rows as context (no prefill on either side): 1 page, 32 pages (four per CTA: two
    groups) and 40 pages with a ragged last page (five per CTA); logits and attention outputs of every
    node against the oracle's tree-masked pass.  cluster = 0: the kernel-per-step path on the same inputs (its
    attention kernel cuts one sequence's pages into four parts up to 1536 tokens and into eight beyond)."""
    import torch
    import paper_2410_21951_b200 as P
    wl = _wide_toy(64, heads=8, tree_caps=(10, 5, 3), index=41)
    w = W.make_weights(wl.shape, wl.seed())
    model = O.Model.from_shape(wl.shape, w)
    N = wl.tree_nodes
    tpl = W.static_template(N, wl.tree_caps)
    g, table = make_gpu(wl.shape, w, 1, N, [ctx_len + N + 8], wl.seed(1))
    g.set_fused_pass(cluster)
    g.begin(table, ctx_len=[ctx_len])
    g.set_tree(tpl.parent, tpl.rank)
    rng = np.random.default_rng(wl.seed(2) + ctx_len)
    g.kv_view().normal_()
    K = O.round_bf16(rng.standard_normal((model.L, ctx_len, model.H, model.dh)))
    V = O.round_bf16(rng.standard_normal((model.L, ctx_len, model.H, model.dh)))
    inject_kv(g, table, 0, K, V)
    kv = O.KVCache(model, capacity=ctx_len + 80)
    kv.extend(K, V)
    toks = rng.integers(0, wl.shape.vocab - 1, size=(1, N)).astype(np.int32)
    logits = torch.zeros(1, N, wl.shape.vocab, dtype=torch.float32, device=g.dev)
    attn = torch.zeros(model.L, 1, N, model.d, dtype=g.tdtype, device=g.dev)
    g.verify_step(override=torch.from_numpy(toks).to(g.dev), logits_out=logits, attn_tap=attn)
    mask = np.zeros((N, N), dtype=bool)
    for n in range(N):
        mask[n, tpl.node_path(n)] = True
    out = O.forward_tree(model, kv, [0] * N, toks[0], ctx_len + tpl.depth, mask)
    lg = logits.cpu().numpy().astype(np.float64)[0]
    at = attn.float().cpu().numpy().astype(np.float64)[:, 0]
    e_l = np.abs(lg - out.logits).max()
    e_a = max(np.abs(at[l] - out.attn[l]).max() for l in range(model.L))
    print(f"context {ctx_len}: max |logit err| {e_l:.2e}, max |attn err| {e_a:.2e}")
    assert e_l <= TOL["bf16"] and e_a <= TOL["bf16"]
    assert cluster == 0 or g.fused_pass_clusters() >= 8
    g.check()
