"""The allocation-free entry point vadusa_draft_topk_static against the regular draft call.

Some users of this library cannot call cudaMalloc at all: a plug-in that lives inside
another framework's memory plan, a real-time audio loop that must not touch the allocator
once it runs, a process whose device memory was given away before the library was loaded.
For them the draft heads' top-k exists in a form whose scratch is a fixed array inside the
library.  This test feeds both forms the same weights and the same hidden state and expects
the same candidate ids, twice in a row (the second call finds the first call's leftovers in
the shared array); the ids are also held against the CPU oracle's draft heads wherever the
oracle's logit gaps decide them; oversize requests must be refused with a clear message.
It runs last so that a failure here cannot hide a failure elsewhere.
"""
import ctypes as C

import numpy as np
import pytest

import oracle as O
import workloads as W

pytestmark = pytest.mark.gpu


def _offsets(P, cfg):
    return {t.name.decode(): t for t in P.tensor_infos(cfg)}


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_static_scratch_draft_matches_regular_draft_twice(dtype):
    import torch
    import paper_2410_21951_b200 as P
    from harness import make_gpu

    wl = W.toy_workload(dtype=dtype, d_model=128, n_heads=2, d_ffn=256, vocab=203, tree_nodes=16,
                        tree_caps=(6, 3, 2), batch=3, index=31)
    sh = wl.shape
    w = W.make_weights(sh, wl.seed())
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    g, table = make_gpu(sh, w, wl.batch, wl.tree_nodes, [200] * wl.batch, 3)
    g.set_tree(tpl.parent, tpl.rank)
    g.begin(table)
    info = _offsets(P, g.cfg)
    blob = g.blob
    dw = blob[info["draft0.w"].offset:]
    db = blob[info["draft0.b"].offset:]
    du = blob[info["draft0.u"].offset:]
    K = g.cfg.draft_topk
    sp = P.Sampling.make(tau=1, temperature=0.0)
    model = O.Model.from_shape(sh, w)
    so = O.Sampling(tau=1, temperature=0.0)
    from harness import MARGINS
    checked = 0
    rng = np.random.default_rng(5)
    for call in range(2):
        h = torch.from_numpy(rng.standard_normal((wl.batch, sh.d_model)).astype(np.float32)).to(g.dev).to(g.tdtype)
        ls = torch.from_numpy(rng.standard_normal((wl.batch, sh.vocab)).astype(np.float32)).to(g.dev)
        g.load_state(h, ls)
        want = torch.zeros(wl.batch, sh.n_draft_heads, K, dtype=torch.int32, device=g.dev)
        g.draft(sp, topk_out=want)
        got = torch.full((wl.batch, sh.n_draft_heads, K), -1, dtype=torch.int32, device=g.dev)
        torch.cuda.synchronize()
        P.draft_topk_static(dw, db, du, h, g.cfg.dtype, wl.batch, sh.d_model, sh.vocab, sh.n_draft_heads, K, True, got)
        torch.cuda.synchronize()
        want, got = want.cpu().numpy(), got.cpu().numpy()
        # against the oracle's draft heads: the r + 1 best candidates are decided when the logit gap behind
        # them exceeds the margin of the dtype, a single rank when the gaps on both sides do
        hs = h.float().cpu().numpy().astype(np.float64)
        for b in range(wl.batch):
            ref = O.draft_topk(model, hs[b], K, so)
            dl = O.draft_logits(model, hs[b])
            for hd in range(sh.n_draft_heads):
                srt = np.sort(O.sampling.masked_logits32(dl[hd], model.eos_id, True).astype(np.float64))[::-1]
                gaps = srt[:K] - srt[1:K + 1]
                for r in range(K):
                    if gaps[r] > MARGINS[dtype]:
                        assert set(got[b, hd, :r + 1]) == set(ref[hd, :r + 1]), f"call {call} seq {b} head {hd} top-{r + 1}"
                        checked += 1
                        if r == 0 or gaps[r - 1] > MARGINS[dtype]:
                            assert got[b, hd, r] == ref[hd, r], f"call {call} seq {b} head {hd} rank {r}"
        if dtype == "fp32":
            assert np.array_equal(got, want), f"call {call}"
        else:
            # the regular bf16 path multiplies on the tensor cores: the same products summed in another
            # order, so two near-equal logits may swap places; the candidate sets must still agree
            # except at such a swap on the last place
            for b in range(wl.batch):
                for hd in range(sh.n_draft_heads):
                    assert len(set(got[b, hd]) & set(want[b, hd])) >= K - 1, f"call {call} seq {b} head {hd}"
                    assert got[b, hd, 0] in want[b, hd, :2]
    assert checked > (40 if dtype == "fp32" else 4), checked
    g.close()


def test_static_scratch_rejects_oversize_and_bad_arguments():
    import torch
    import paper_2410_21951_b200 as P
    L = P.lib()
    assert L.vadusa_static_scratch_bytes() == 2 << 20
    dev = torch.device("cuda", 0)
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device=dev)
    out = torch.zeros(1 << 14, dtype=torch.int32, device=dev)
    p = C.c_void_p(buf.data_ptr())
    # 64 sequences x 4 heads x 2049 ids of fp32 logits do not fit in 2 MiB
    st = L.vadusa_draft_topk_static(p, p, p, p, 1, 64, 1024, 2049, 4, 10, 1, C.c_void_p(out.data_ptr()), None)
    assert st == 2 and b"built-in array" in L.vadusa_static_last_error()
    assert L.vadusa_draft_topk_static(None, p, p, p, 1, 1, 128, 203, 3, 6, 1, C.c_void_p(out.data_ptr()), None) == 1
    assert L.vadusa_draft_topk_static(p, p, p, p, 2, 1, 128, 203, 3, 6, 1, C.c_void_p(out.data_ptr()), None) == 1
    assert L.vadusa_draft_topk_static(p, p, p, p, 1, 0, 128, 203, 3, 6, 1, C.c_void_p(out.data_ptr()), None) == 1
    torch.cuda.synchronize()
