"""Pins of the oracle's model against things other than itself: torch's own
transformer encoder layer, torch's bf16 conversion, tree-mask semantics against
path-only passes, and chain trees against an ordinary causal pass."""
import json
import os

import numpy as np
import pytest
import torch

import oracle as O
import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _toy(dtype="fp32", **kw):
    wl = W.toy_workload(dtype=dtype, **kw)
    w = W.make_weights(wl.shape, wl.seed())
    return wl, w, O.Model.from_shape(wl.shape, w)


def test_bf16_rounding_matches_torch_conversion():
    g = np.random.default_rng(0)
    x = np.concatenate([g.standard_normal(20000) * 10.0 ** g.integers(-6, 6, 20000),
                        [1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 3 * 2.0 ** -8, 0.0, -0.0]])
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x), ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert O.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    # workloads' own rounding of weights agrees
    assert np.array_equal(W.round_to_bf16_values(x.astype(np.float32)).astype(np.float64), ref)


def test_forward_token_matches_torch_transformer_encoder():
    """The path-only pass over a sequence equals torch.nn.TransformerEncoder
    (norm_first, ReLU) under a causal mask, position by position."""
    wl, w, m = _toy(n_layers=3)
    sh = wl.shape
    layer = torch.nn.TransformerEncoderLayer(sh.d_model, sh.n_heads, sh.d_ffn, dropout=0.0,
                                             activation="relu", batch_first=True, norm_first=True,
                                             layer_norm_eps=sh.ln_eps, dtype=torch.float64)
    enc = torch.nn.TransformerEncoder(layer, sh.n_layers, enable_nested_tensor=False)
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    with torch.no_grad():
        for l, lyr in enumerate(enc.layers):
            p = f"l{l}."
            lyr.self_attn.in_proj_weight.copy_(t(w[p + "wqkv"])); lyr.self_attn.in_proj_bias.copy_(t(w[p + "bqkv"]))
            lyr.self_attn.out_proj.weight.copy_(t(w[p + "wo"])); lyr.self_attn.out_proj.bias.copy_(t(w[p + "bo"]))
            lyr.linear1.weight.copy_(t(w[p + "w1"])); lyr.linear1.bias.copy_(t(w[p + "b1"]))
            lyr.linear2.weight.copy_(t(w[p + "w2"])); lyr.linear2.bias.copy_(t(w[p + "b2"]))
            lyr.norm1.weight.copy_(t(w[p + "ln1_g"])); lyr.norm1.bias.copy_(t(w[p + "ln1_b"]))
            lyr.norm2.weight.copy_(t(w[p + "ln2_g"])); lyr.norm2.bias.copy_(t(w[p + "ln2_b"]))
    enc.eval()
    ph, pr = W.prefix_for(wl, 0)
    T = len(ph) + len(pr)
    x = torch.stack([t(w["emb_phon"][p]) for p in ph] + [t(w["emb_audio"][a]) for a in pr]) + t(w["pos"][:T])
    causal = torch.triu(torch.ones(T, T, dtype=torch.bool), diagonal=1)
    with torch.no_grad():
        y = enc(x[None], mask=causal)[0]
        y = torch.nn.functional.layer_norm(y, (sh.d_model,), t(w["lnf_g"]), t(w["lnf_b"]), sh.ln_eps)
        ref_logits = (y @ t(w["lm"]).T).numpy()
    kv = O.KVCache(m)
    pos = 0
    for p in ph:
        out = O.forward_token(m, kv, 1, int(p), pos)
        assert np.allclose(out.logits, ref_logits[pos], atol=1e-10); pos += 1
    for a in pr:
        out = O.forward_token(m, kv, 0, int(a), pos)
        assert np.allclose(out.logits, ref_logits[pos], atol=1e-10); pos += 1
    assert np.allclose(out.h, y[-1].numpy(), atol=1e-10)


def test_draft_head_matches_torch_functional():
    wl, w, m = _toy()
    g = np.random.default_rng(1)
    h = g.standard_normal(wl.shape.d_model)
    got = O.draft_logits(m, h)
    ht = torch.tensor(h)
    for i in range(wl.shape.n_draft_heads):
        t = torch.nn.functional.linear(ht, torch.tensor(w[f"draft{i}.w"], dtype=torch.float64),
                                       torch.tensor(w[f"draft{i}.b"], dtype=torch.float64))
        z = ht + torch.nn.functional.silu(t)
        ref = torch.nn.functional.linear(z, torch.tensor(w[f"draft{i}.u"], dtype=torch.float64)).numpy()
        assert np.allclose(got[i], ref, atol=1e-12)


@pytest.mark.parametrize("dtype,tol", [("fp32", 1e-10), ("bf16", 3e-2)])
def test_tree_masked_scores_equal_path_only_scores(dtype, tol):
    """Sec. II-A: with the tree-attention mask the whole tree is verified in one
    pass; every node's scores must equal those of its own root path fed alone."""
    wl, w, m = _toy(dtype=dtype)
    ph, pr = W.prefix_for(wl, 0)
    st = O.prefill(m, ph, pr)
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    g = np.random.default_rng(2)
    toks = g.integers(0, wl.shape.vocab - 1, tpl.n_nodes)
    N = tpl.n_nodes
    mask = np.zeros((N, N), dtype=bool)
    for n in range(N):
        mask[n, tpl.node_path(n)] = True
    tree = O.forward_tree(m, st.kv, [0] * N, toks, st.S + tpl.depth, mask)
    for n in range(N):
        bkv = st.kv.branch()
        for i, a in enumerate(tpl.node_path(n)):
            out = O.forward_token(m, bkv, 0, int(toks[a]), st.S + i, taps=True)
        assert np.abs(out.logits - tree.logits[n]).max() < tol
        assert np.abs(out.h - tree.h[n]).max() < (tol if dtype == "fp32" else 0.07)
        for l in range(m.L):
            assert np.abs(out.attn[l] - tree.attn[l][n]).max() < tol
    # a wrong mask (a node also sees a sibling) must change the scores
    bad = mask.copy(); bad[2, 1] = True
    worse = O.forward_tree(m, st.kv, [0] * N, toks, st.S + tpl.depth, bad)
    assert np.abs(worse.logits[2] - tree.logits[2]).max() > 1e-6


def test_chain_tree_is_a_causal_pass_and_blocked_prefill_agrees():
    wl, w, m = _toy()
    ph, pr = W.prefix_for(wl, 0)
    a = O.prefill(m, ph, pr)
    for chunk in (1, 4, 5, 64):
        b = O.prefill_blocked(m, ph, pr, chunk=chunk)
        assert np.allclose(a.logits_star, b.logits_star, atol=1e-11)
        assert np.allclose(a.kv.K[:, :a.S], b.kv.K[:, :b.S], atol=1e-11)
        assert np.allclose(a.kv.V[:, :a.S], b.kv.V[:, :b.S], atol=1e-11)
        assert a.S == b.S == len(ph) + len(pr)


def test_branch_cache_does_not_leak_into_parent():
    wl, w, m = _toy()
    ph, pr = W.prefix_for(wl, 0)
    st = O.prefill(m, ph, pr)
    n0, K0 = st.kv.n, st.kv.K.copy()
    b = st.kv.branch()
    O.forward_token(m, b, 0, 3, st.S)
    assert st.kv.n == n0 and b.n == n0 + 1 and np.array_equal(st.kv.K, K0)


def test_table1_context_numbers():
    rows = json.load(open(os.path.join(GOLDEN, "table1_ratios.json")))["rows"]
    for r in rows:
        assert 1.0 <= r["acc"] <= 5.0                      # 4 heads: at most root + 4 drafts
        assert 1.15 < r["acc"] / r["speedup"] < 1.35       # a tree pass costs 1.2-1.3 AR steps
