"""Decoding loops of the oracle (test infrastructure only).

`ar_decode` is plain one-token-at-a-time decoding.  `vadusa_iteration` is one
draft-and-verify iteration as the paper states it (Sec. II-A, II-C): the base
head gives the root, draft head i fills depth i of the candidate tree with its
top-k tokens, every root-to-leaf branch is scored by its own sequential causal
pass and checked with Algorithm 1, the longest (then leftmost) accepted branch
is kept, and decoding continues from the base head's distribution at the last
accepted token.

End of sequence (the paper does not treat it; its tolerance-1 decoding is lossless,
Sec. II-A, so nothing may follow a token at which plain decoding would have stopped):
with `eos_masked` the EOS id can never be drawn or drafted and generation ends by
length; without it, a sequence is finished as soon as EOS is committed, and the
tokens behind EOS on the accepted path are dropped.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

from .model import AUDIO, PHONEME, KVCache, Model, draft_logits, forward_token, forward_tree
from .sampling import (decision_keys, masked_logits32, nucleus_mass_before, nucleus_sorted,
                       root_token, sample_set, topk_ids)
from .verify import select_best, verify_branch


@dataclass(frozen=True)
class Sampling:
    tau: int = 1
    temperature: float = 0.0      # 0: greedy
    top_p: float = 1.0            # >= 1: nucleus off
    eos_masked: bool = True
    accept_rule: int = 0          # 0: Alg. 1 (tau noisy draws); 1: plain top-tau of the logits
    seed: int = 0
    bias: Optional[np.ndarray] = None   # [sequences][vocab] fp32 added to the base head's logits wherever it samples


@dataclass
class State:
    kv: KVCache
    tokens: List[int]             # generated tokens so far
    h_star: np.ndarray            # final hidden state at the last committed token
    logits_star: np.ndarray       # base-head logits there (they predict position kv.n)
    seq: int = 0                  # sequence id, enters the noise only
    finished: bool = False        # EOS has been committed (only when EOS is not masked)

    @property
    def S(self) -> int:
        return self.kv.n


def prefill(model: Model, phon: Sequence[int], prompt: Sequence[int], seq: int = 0) -> State:
    """Feed [phonemes ; prompt tokens] one by one with a running position index."""
    kv = KVCache(model, capacity=len(phon) + len(prompt) + 64)
    out = None
    pos = 0
    for t in phon:
        out = forward_token(model, kv, PHONEME, int(t), pos); pos += 1
    for t in prompt:
        out = forward_token(model, kv, AUDIO, int(t), pos); pos += 1
    return State(kv=kv, tokens=[], h_star=out.h, logits_star=out.logits, seq=seq)


def prefill_blocked(model: Model, phon: Sequence[int], prompt: Sequence[int], seq: int = 0,
                    chunk: int = 128) -> State:
    """Same state as `prefill`, computed chunk by chunk with `forward_tree` under a
    lower-triangular mask (a chain-shaped tree is an ordinary causal pass)."""
    kinds = [PHONEME] * len(phon) + [AUDIO] * len(prompt)
    toks = [int(t) for t in phon] + [int(t) for t in prompt]
    kv = KVCache(model, capacity=len(toks) + 64)
    out = None
    for s in range(0, len(toks), chunk):
        e = min(len(toks), s + chunk)
        mask = np.tril(np.ones((e - s, e - s), dtype=bool))
        out = forward_tree(model, kv, kinds[s:e], toks[s:e], list(range(s, e)), mask)
        kv.extend(out.K, out.V)
    return State(kv=kv, tokens=[], h_star=out.h[-1], logits_star=out.logits[-1], seq=seq)


def _keys_and_nucleus(model: Model, logits, sp: Sampling, seq: int, pos: int, noise: bool = True):
    l32 = masked_logits32(logits, model.eos_id, sp.eos_masked)
    if sp.bias is not None:
        # a reshaped base-head distribution (Sec. II-C, last paragraph: other sampling strategies enter as the
        # original head's predictions): one fp32 addition before temperature, nucleus and noise
        l32 = (l32 + np.asarray(sp.bias[seq], dtype=np.float32)).astype(np.float32)
    keys = decision_keys(l32, sp.temperature, sp.seed, seq, pos, noise=noise)
    nuc = nucleus_sorted(l32, sp.temperature, sp.top_p)
    return l32, keys, nuc


def sample_next(model: Model, logits, sp: Sampling, seq: int, pos: int) -> int:
    """The base head's single sample for absolute position `pos`."""
    _, keys, nuc = _keys_and_nucleus(model, logits, sp, seq, pos)
    return root_token(keys, nuc)


def draws_at(model: Model, logits, sp: Sampling, seq: int, pos: int) -> List[int]:
    """v: the tau draws of Alg. 1 line 3 for the token at absolute position `pos`."""
    _, keys, nuc = _keys_and_nucleus(model, logits, sp, seq, pos, noise=(sp.accept_rule == 0))
    return sample_set(keys, nuc, sp.tau)


def ar_decode(model: Model, st: State, sp: Sampling, n_tokens: int) -> List[int]:
    """Plain AR decoding from state `st` (which is advanced)."""
    out = []
    for _ in range(n_tokens):
        if st.finished:
            break
        pos = st.S
        tok = sample_next(model, st.logits_star, sp, st.seq, pos)
        if not sp.eos_masked and tok == model.eos_id:
            st.finished = True
        r = forward_token(model, st.kv, AUDIO, tok, pos)
        st.h_star, st.logits_star = r.h, r.logits
        st.tokens.append(tok); out.append(tok)
    return out


def draft_topk(model: Model, h_star, k: int, sp: Sampling) -> np.ndarray:
    """[n_draft, k] ids: the k largest logits of every draft head at h_star."""
    dl = draft_logits(model, h_star)
    return np.stack([topk_ids(masked_logits32(dl[i], model.eos_id, sp.eos_masked), k)
                     for i in range(model.n_draft)])


def build_tree_tokens(template, root: int, topk: np.ndarray) -> np.ndarray:
    """Node 0 holds the root; a node of depth d >= 1 holds candidate number rank[n]
    of draft head d (Sec. II-A: layer i+1 of the tree is filled from head i)."""
    toks = np.zeros(template.n_nodes, dtype=np.int32)
    toks[0] = root
    for n in range(1, template.n_nodes):
        toks[n] = topk[int(template.depth[n]) - 1, int(template.rank[n])]
    return toks


@dataclass
class IterationTrace:
    S: int
    root: int
    topk: np.ndarray
    tree_tokens: np.ndarray
    node_logits: np.ndarray          # [N, V] float64, NaN rows for nodes that were not scored
    node_h: np.ndarray               # [N, d]
    edge_ok: np.ndarray              # [N] bool (edge parent -> node accepted); [0] True
    accept_len: int
    best_node: int
    path_nodes: List[int]
    path_tokens: List[int]
    margin_root: float
    margin_draft: np.ndarray         # [n_draft]
    draft_gaps: np.ndarray           # [n_draft, kmax]: logit gap between candidates r and r+1 of each head
    margin_accept: float
    attn: Optional[List[np.ndarray]] = None     # per layer [N, d]: attention output (before the output projection)
    K: Optional[np.ndarray] = None              # [L, N, H, dh] rows of every node (tree/memo mode)
    V: Optional[np.ndarray] = None
    finished: bool = False                      # EOS was committed in this iteration


def _gap_top2(keys, nuc) -> float:
    k = np.sort(keys[nuc].astype(np.float64))[::-1]
    return float(k[0] - k[1]) if k.shape[0] > 1 else float("inf")


def _draft_margin(l32: np.ndarray, n_used: int) -> float:
    """Smallest gap between neighbours among the n_used+1 largest logits."""
    k = np.sort(l32.astype(np.float64))[::-1][: n_used + 1]
    return float(np.min(k[:-1] - k[1:])) if k.shape[0] > 1 else float("inf")


def _edge_margin(model: Model, logits, sp: Sampling, seq: int, pos: int, c: int) -> float:
    """Distance of candidate c from the boundary of the draw set at one node."""
    l32, keys, nuc = _keys_and_nucleus(model, logits, sp, seq, pos, noise=(sp.accept_rule == 0))
    m = float("inf")
    if sp.temperature != 0.0 and sp.top_p < 1.0:
        # how close any prefix mass of the descending-probability order comes to top_p:
        # the membership of every token, not only of c, shapes the draw set
        z = l32.astype(np.float64) / float(sp.temperature)
        p = np.exp(z - z.max()); p = np.sort(p / p.sum())[::-1]
        before = np.concatenate([[0.0], np.cumsum(p)[:-1]])
        m = float(np.min(np.abs(before - sp.top_p)))
    if not nuc[c]:
        return m
    ks = np.sort(keys[nuc].astype(np.float64))[::-1]
    inside = c in sample_set(keys, nuc, sp.tau)
    if inside:
        if ks.shape[0] > sp.tau:
            m = min(m, float(keys[c]) - ks[sp.tau])
    else:
        m = min(m, ks[sp.tau - 1] - float(keys[c]))
    return m


def vadusa_iteration(model: Model, st: State, template, sp: Sampling, mode: str = "branch",
                     tokens_override: Optional[np.ndarray] = None,
                     forced_best: Optional[int] = None, taps: bool = False) -> IterationTrace:
    """One draft-and-verify iteration; advances `st` by the accepted tokens.

    mode "branch": every root-to-leaf branch gets its own sequential pass over a
    copy of the committed cache (the defining mode).  mode "memo": each node is
    fed once, after the stored K/V rows of its ancestors (same arithmetic, fewer
    passes).  mode "tree": all nodes in one `forward_tree` pass under the
    ancestor mask."""
    S, seq, N = st.S, st.seq, template.n_nodes
    kmax = int(template.rank.max()) + 1
    l32s, keys_s, nuc_s = _keys_and_nucleus(model, st.logits_star, sp, seq, S)
    root = root_token(keys_s, nuc_s)
    topk = draft_topk(model, st.h_star, kmax, sp)
    dl = draft_logits(model, st.h_star)
    margin_draft = np.array([
        _draft_margin(masked_logits32(dl[i], model.eos_id, sp.eos_masked),
                      int(template.rank[template.depth == i + 1].max()) + 1 if np.any(template.depth == i + 1) else 0)
        for i in range(model.n_draft)])
    draft_gaps = np.zeros((model.n_draft, kmax))
    for i in range(model.n_draft):
        srt = np.sort(masked_logits32(dl[i], model.eos_id, sp.eos_masked).astype(np.float64))[::-1]
        draft_gaps[i] = srt[:kmax] - srt[1:kmax + 1]
    toks = build_tree_tokens(template, root, topk) if tokens_override is None \
        else np.asarray(tokens_override, dtype=np.int32).copy()

    node_logits = np.full((N, model.V), np.nan)
    node_h = np.full((N, model.d), np.nan)
    node_K = np.zeros((model.L, N, model.H, model.dh)); node_V = np.zeros_like(node_K)
    have = np.zeros(N, dtype=bool)
    attn = [np.zeros((N, model.d)) for _ in range(model.L)]      # per layer: attention output of every node

    def record(n, out, K1, V1):
        if have[n]:
            assert np.array_equal(node_logits[n], out.logits), "a node's scores depend on the branch"
        node_logits[n], node_h[n] = out.logits, out.h
        node_K[:, n], node_V[:, n] = K1[:, 0], V1[:, 0]
        for l in range(model.L):
            attn[l][n] = out.attn[l]
        have[n] = True

    leaves = template.leaves()
    if mode == "branch":
        for leaf in leaves:
            bkv = st.kv.branch()
            for i, n in enumerate(template.node_path(leaf)):
                out = forward_token(model, bkv, AUDIO, int(toks[n]), S + i, taps=True)
                record(n, out, *bkv.own_rows(i, 1))
    elif mode == "memo":
        for n in range(N):
            path = template.node_path(n)
            bkv = st.kv.branch()
            if len(path) > 1:
                bkv.extend(node_K[:, path[:-1]], node_V[:, path[:-1]])
            out = forward_token(model, bkv, AUDIO, int(toks[n]), S + len(path) - 1, taps=True)
            record(n, out, *bkv.own_rows(len(path) - 1, 1))
    elif mode == "tree":
        mask = np.zeros((N, N), dtype=bool)
        for n in range(N):
            mask[n, template.node_path(n)] = True
        out = forward_tree(model, st.kv, [AUDIO] * N, toks, S + template.depth, mask)
        node_logits, node_h, node_K, node_V = out.logits, out.h, out.K, out.V
        attn = out.attn
        have[:] = True
    else:
        raise ValueError(mode)

    # Alg. 1 on every branch: v_i is drawn from the logits at candidate i, which
    # predict absolute position S + i + 1.
    draws: Dict[int, List[int]] = {}

    def v_of(n):
        if n not in draws:
            draws[n] = draws_at(model, node_logits[n], sp, seq, S + int(template.depth[n]) + 1)
        return draws[n]

    results = []
    for leaf in leaves:
        path = template.node_path(leaf)
        cands = [int(toks[n]) for n in path]
        sets = [v_of(n) for n in path[:-1]] + [[]]
        results.append((template.rank_path(leaf), verify_branch(cands, sets)))
    win = select_best(results)
    k_star = results[win][1]
    path = template.node_path(leaves[win])[: k_star + 1]
    if forced_best is not None:
        path = template.node_path(int(forced_best))
        k_star = len(path) - 1
    finished = False
    if not sp.eos_masked:
        for j, n in enumerate(path):
            if int(toks[n]) == model.eos_id:          # the sequence ends here: drop what follows EOS
                path, k_star, finished = path[: j + 1], j, True
                break
    best = path[-1]

    edge_ok = np.zeros(N, dtype=bool); edge_ok[0] = True
    for n in range(1, N):
        edge_ok[n] = int(toks[n]) in v_of(int(template.parent[n]))
    accepted = np.zeros(N, dtype=bool); accepted[0] = True
    margin_accept = float("inf")
    for n in range(1, N):
        p = int(template.parent[n])
        accepted[n] = accepted[p] and edge_ok[n]
        if accepted[p]:
            margin_accept = min(margin_accept, _edge_margin(
                model, node_logits[p], sp, seq, S + int(template.depth[p]) + 1, int(toks[n])))

    st.kv.extend(node_K[:, path], node_V[:, path])
    st.tokens.extend(int(toks[n]) for n in path)
    st.h_star, st.logits_star = node_h[best].copy(), node_logits[best].copy()
    st.finished = st.finished or finished
    return IterationTrace(S=S, root=root, topk=topk, tree_tokens=toks, node_logits=node_logits,
                          node_h=node_h, edge_ok=edge_ok, accept_len=k_star + 1, best_node=best,
                          path_nodes=list(path), path_tokens=[int(toks[n]) for n in path],
                          margin_root=_gap_top2(keys_s, nuc_s), margin_draft=margin_draft, draft_gaps=draft_gaps,
                          margin_accept=margin_accept, attn=attn, K=node_K, V=node_V, finished=finished)


def vadusa_generate(model: Model, st: State, template, sp: Sampling, n_tokens: int,
                    mode: str = "branch", max_iters: Optional[int] = None) -> List[IterationTrace]:
    """Iterate until at least n_tokens have been generated (or max_iters, or EOS committed)."""
    traces = []
    start = len(st.tokens)
    while (len(st.tokens) - start < n_tokens and (max_iters is None or len(traces) < max_iters)
           and not st.finished):
        traces.append(vadusa_iteration(model, st, template, sp, mode=mode))
    return traces
