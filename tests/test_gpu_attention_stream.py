"""The page-stream attention kernel for batches (one persistent kernel over the K/V pages of all
(sequence, head) pairs; paper Sec. II-A, tree attention) against the CPU oracle, on ragged batches built
so that pairs are cut at thread-block boundaries in every way the kernel distinguishes: whole pairs,
pairs in two parts, one pair spread over many blocks, sequences of one page, sequences that have ended.
The same passes also run through the kernel with one thread block per (head, sequence); the two must agree."""
import numpy as np
import pytest

import oracle as O
import workloads as W
from harness import TOL, inject_kv, make_gpu

pytestmark = pytest.mark.gpu


def _mask(tpl):
    N = tpl.n_nodes
    m = np.zeros((N, N), dtype=bool)
    for n in range(N):
        m[n, tpl.node_path(n)] = True
    return m


def _context(model, S, rng):
    K = O.round_bf16(rng.standard_normal((model.L, S, model.H, model.dh)))
    V = O.round_bf16(rng.standard_normal((model.L, S, model.H, model.dh)))
    return K, V


@pytest.mark.parametrize("nodes,per_seq,lens_kind", [(64, True, "one_long"), (42, False, "short"), (64, False, "two_long")])
def test_page_stream_attention_on_ragged_batches(nodes, per_seq, lens_kind):
    import torch
    B = 80                                                   # 160 (sequence, head) pairs: more than one per SM
    wl = W.toy_workload(dtype="bf16", n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=203, tree_nodes=nodes,
                        tree_caps=(10, 5, 3), batch=B, index=61, max_pos=4096)
    sh = wl.shape
    w = W.make_weights(sh, wl.seed())
    model = O.Model.from_shape(sh, w)
    rng = np.random.default_rng(wl.seed(3))
    if lens_kind == "one_long":
        # one sequence holds most of the pages: its two pairs are spread over many thread blocks
        lens = rng.integers(1, 130, size=B).astype(np.int32)
        lens[7] = 2500
    elif lens_kind == "two_long":
        lens = rng.integers(40, 400, size=B).astype(np.int32)
        lens[0], lens[B - 1] = 1900, 1300                    # the first and the last pair of the stream are long
    else:
        lens = rng.integers(1, 64 - nodes + 1, size=B).astype(np.int32)   # context and tree within one page
        lens[5:9] = [64, 65, 63 - nodes + 64, 200]
    g, table = make_gpu(sh, w, B, nodes, [int(s) + nodes + 8 for s in lens], wl.seed(1))
    if per_seq:
        tpls = [W.random_topology(nodes, sh.n_draft_heads, wl.seed(100 + b)) for b in range(B)]
    else:
        tpls = [W.static_template(nodes, wl.tree_caps)] * B

    def begin():
        g.begin(table, ctx_len=lens)
        if per_seq:                                          # per-sequence trees belong to one batch: set again
            g.set_tree(np.stack([t.parent for t in tpls]), np.stack([t.rank for t in tpls]), per_sequence=True)
        else:
            g.set_tree(tpls[0].parent, tpls[0].rank)

    begin()
    g.kv_view().normal_()
    caches = {}
    for b in range(B):
        K, V = _context(model, int(lens[b]), rng)
        inject_kv(g, table, b, K, V)
        kv = O.KVCache(model, capacity=int(lens[b]) + nodes + 8)
        kv.extend(K, V)
        caches[b] = kv
    toks = rng.integers(0, sh.vocab - 1, size=(B, nodes)).astype(np.int32)
    dev_toks = torch.from_numpy(toks).to(g.dev)
    taps, lgs = {}, {}
    for stream in (True, False):
        g.set_attention_stream(stream)
        logits = torch.zeros(B, nodes, sh.vocab, dtype=torch.float32, device=g.dev)
        attn = torch.zeros(model.L, B, nodes, model.d, dtype=g.tdtype, device=g.dev)
        begin()
        g.verify_step(override=dev_toks, logits_out=logits, attn_tap=attn)
        g.check()
        taps[stream] = attn.float().cpu().numpy().astype(np.float64)
        lgs[stream] = logits.cpu().numpy().astype(np.float64)
        if stream:
            # once more from the same state: the counters of the merged pairs are back at zero, and whichever
            # part of a pair arrives last, the parts are summed in the same order: bit-identical outputs
            attn2 = torch.zeros_like(attn)
            begin()
            g.verify_step(override=dev_toks, attn_tap=attn2)
            g.check()
            assert torch.equal(attn, attn2)
    worst_a = worst_l = 0.0
    for b in range(B):
        tpl = tpls[b]
        out = O.forward_tree(model, caches[b], [0] * nodes, toks[b], int(lens[b]) + tpl.depth, _mask(tpl))
        for stream in (True, False):
            e_a = max(np.abs(taps[stream][l, b] - out.attn[l]).max() for l in range(model.L))
            e_l = np.abs(lgs[stream][b] - out.logits).max()
            assert e_a <= TOL["bf16"] and e_l <= TOL["bf16"], f"seq {b} (context {int(lens[b])}) stream={stream}: {e_a:.2e} {e_l:.2e}"
            if stream:
                worst_a, worst_l = max(worst_a, e_a), max(worst_l, e_l)
    # the two kernels round at the same points per page and differ only in how partial sums are merged
    d = np.abs(taps[True] - taps[False]).max()
    print(f"page-stream attention, {lens_kind}: max |attn err| {worst_a:.2e}, max |logit err| {worst_l:.2e}, "
          f"max |stream - per-sequence| {d:.2e}")
    assert d <= 1.6e-2
    g.close()


def test_page_stream_attention_leaves_ended_sequences_alone():
    """Sequences that have ended (no tree) have no pages in the stream: their output rows are zero, and the
    rows of the others are what they are without them."""
    import torch
    import paper_2410_21951_b200 as P
    B, nodes = 80, 16
    wl = W.toy_workload(dtype="bf16", n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=203, tree_nodes=nodes,
                        tree_caps=(6, 3, 2), batch=B, index=62, max_pos=1024)
    sh = wl.shape
    w = W.make_weights(sh, wl.seed())
    model = O.Model.from_shape(sh, w)
    tpl = W.static_template(nodes, wl.tree_caps)
    rng = np.random.default_rng(wl.seed(3))
    lens = rng.integers(30, 300, size=B).astype(np.int32)
    g, table = make_gpu(sh, w, B, nodes, [int(s) + 3 * nodes for s in lens], wl.seed(1))
    g.set_tree(tpl.parent, tpl.rank)
    g.begin(table, ctx_len=lens)
    g.kv_view().normal_()
    caches = {}
    for b in range(B):
        K, V = _context(model, int(lens[b]), rng)
        inject_kv(g, table, b, K, V)
        kv = O.KVCache(model, capacity=int(lens[b]) + 3 * nodes)
        kv.extend(K, V)
        caches[b] = kv
    # first iteration: EOS (not masked) forced as the root's child of every third sequence, which ends there
    eos = sh.vocab - 1
    sg = P.Sampling.make(tau=1, temperature=0.0, eos_masked=0)
    toks = rng.integers(0, sh.vocab - 1, size=(B, nodes)).astype(np.int32)
    ended = np.arange(B) % 3 == 1
    child = int(np.nonzero(tpl.depth == 1)[0][0])
    toks[ended, child] = eos
    forced = torch.full((B,), child, dtype=torch.int32, device=g.dev)
    acc = torch.zeros(B, dtype=torch.int32, device=g.dev)
    g.verify_step(override=torch.from_numpy(toks).to(g.dev))
    g.accept_and_commit(sg, forced_best=forced, accept_len=acc)
    assert np.all(acc.cpu().numpy() == 2)
    lens2 = g.lengths().copy()
    assert np.array_equal(lens2, lens + 2)
    # second iteration over the batch with holes
    toks2 = rng.integers(0, sh.vocab - 1, size=(B, nodes)).astype(np.int32)
    attn = torch.full((model.L, B, nodes, model.d), 7.0, dtype=g.tdtype, device=g.dev)
    logits = torch.zeros(B, nodes, sh.vocab, dtype=torch.float32, device=g.dev)
    g.verify_step(override=torch.from_numpy(toks2).to(g.dev), logits_out=logits, attn_tap=attn)
    g.check()
    at = attn.float().cpu().numpy().astype(np.float64)
    lg = logits.cpu().numpy().astype(np.float64)
    path = tpl.node_path(child)
    checked = 0
    for b in range(B):
        if ended[b]:
            assert np.all(at[:, b] == 0.0), f"ended sequence {b}"
            continue
        if b % 4:
            continue                                         # the oracle follows every fourth live sequence
        out1 = O.forward_tree(model, caches[b], [0] * nodes, toks[b], int(lens[b]) + tpl.depth, _mask(tpl))
        caches[b].extend(out1.K[:, path], out1.V[:, path])
        out = O.forward_tree(model, caches[b], [0] * nodes, toks2[b], int(lens2[b]) + tpl.depth, _mask(tpl))
        e_a = max(np.abs(at[l, b] - out.attn[l]).max() for l in range(model.L))
        e_l = np.abs(lg[b] - out.logits).max()
        assert e_a <= TOL["bf16"] and e_l <= TOL["bf16"], f"seq {b}: {e_a:.2e} {e_l:.2e}"
        checked += 1
    assert checked >= 12
    g.close()
