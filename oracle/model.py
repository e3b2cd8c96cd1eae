"""The speech-token language model of the oracle (test infrastructure only).

A plain pre-LN decoder-only transformer in float64 (Sec. III-A.1 of the paper
gives the sizes: 12 layers, 16 heads each with its own K/V, d 1024, FFN 4096)
with the draft heads of Sec. II-A / III-A.1 (a residual block of one linear
layer and a SiLU, then a vocabulary projection per head).

`forward_token` is the defining routine: one token at a time, attending to all
tokens fed before it, so it is causal by construction and needs no mask.
`forward_tree` is a second, independent routine that scores many nodes in one
pass under an explicit tree mask (Sec. II-A, "tree attention"); it exists to be
checked against `forward_token` and to give taps for large cases.

In a "bf16" model the quantities the model stores in bf16 are rounded (nearest
even) where they are produced: LayerNorm outputs, q/k/v, the attention output,
the feed-forward hidden layer, the final hidden state, and the draft heads'
residual-block output.  Sums and what feeds them without being stored (residual
stream, dot products, softmax weights and denominators, logits) are never
rounded, so the definition does not depend on the order in which keys are
visited.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np

from .numerics import round_bf16

AUDIO, PHONEME = 0, 1


class Model:
    def __init__(self, weights: Dict[str, np.ndarray], n_layers: int, d_model: int, n_heads: int,
                 d_ffn: int, vocab: int, n_draft_heads: int, dtype: str, ln_eps: float = 1e-5):
        self.w = {k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}
        self.L, self.d, self.H, self.F, self.V = n_layers, d_model, n_heads, d_ffn, vocab
        self.dh = d_model // n_heads
        self.n_draft = n_draft_heads
        self.dtype = dtype
        self.eps = ln_eps
        self.scale = 1.0 / np.sqrt(self.dh)
        self.eos_id = vocab - 1

    @classmethod
    def from_shape(cls, shape, weights):
        return cls(weights, shape.n_layers, shape.d_model, shape.n_heads, shape.d_ffn, shape.vocab,
                   shape.n_draft_heads, shape.dtype, shape.ln_eps)

    def R(self, a):
        """Storage rounding of the model: bf16 in a bf16 model, nothing otherwise."""
        return round_bf16(a) if self.dtype == "bf16" else np.asarray(a, dtype=np.float64)

    def layer_norm(self, x, g, b):
        mu = x.mean(axis=-1, keepdims=True)
        var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
        return (x - mu) / np.sqrt(var + self.eps) * g + b

    def embed(self, kind: int, tok: int, pos: int):
        table = self.w["emb_phon"] if kind == PHONEME else self.w["emb_audio"]
        return table[tok] + self.w["pos"][pos]


class KVCache:
    """Keys and values of the tokens fed so far, per layer: arrays [L, n, H, dh].

    `branch()` gives a cache that starts as a logical copy of this one; what is
    appended to the branch does not show in the parent (the parent's rows are
    shared read-only instead of being copied)."""

    def __init__(self, model: Model, capacity: int = 64, parent: Optional["KVCache"] = None):
        self.m = model
        self.parent = parent
        self.base_n = parent.n if parent is not None else 0
        self.K = np.zeros((model.L, capacity, model.H, model.dh))
        self.V = np.zeros((model.L, capacity, model.H, model.dh))
        self.own = 0

    @property
    def n(self) -> int:
        return self.base_n + self.own

    def branch(self) -> "KVCache":
        assert self.parent is None, "branch only from a committed cache"
        return KVCache(self.m, capacity=16, parent=self)

    def _grow(self, need):
        if need > self.K.shape[1]:
            cap = max(need, 2 * self.K.shape[1])
            for name in ("K", "V"):
                old = getattr(self, name)
                new = np.zeros((old.shape[0], cap) + old.shape[2:])
                new[:, :old.shape[1]] = old
                setattr(self, name, new)

    def append(self, layer: int, k, v):
        """Store the K/V of the token being fed at `layer`; the token counts once
        `advance()` is called after its last layer."""
        self._grow(self.own + 1)
        self.K[layer, self.own] = k
        self.V[layer, self.own] = v

    def advance(self):
        self.own += 1

    def rows(self, layer: int, upto_own: int):
        """K, V [t, H, dh] of the first base_n + upto_own tokens."""
        if self.parent is None:
            return self.K[layer, :upto_own], self.V[layer, :upto_own]
        pk, pv = self.parent.rows(layer, self.base_n)
        return (np.concatenate([pk, self.K[layer, :upto_own]], axis=0),
                np.concatenate([pv, self.V[layer, :upto_own]], axis=0))

    def own_rows(self, first: int, count: int):
        """Copies of own rows [first, first+count): (K, V) each [L, count, H, dh]."""
        return self.K[:, first:first + count].copy(), self.V[:, first:first + count].copy()

    def extend(self, K, V):
        """Append `count` finished tokens given as [L, count, H, dh] arrays."""
        c = K.shape[1]
        self._grow(self.own + c)
        self.K[:, self.own:self.own + c] = K
        self.V[:, self.own:self.own + c] = V
        self.own += c


@dataclass
class TokenOut:
    h: np.ndarray             # final-LayerNorm output [d] (bf16-valued in a bf16 model)
    logits: np.ndarray        # base head logits [V], float64
    attn: Optional[List[np.ndarray]] = None   # per layer: attention output [d] (before the output projection)


def forward_token(model: Model, kv: KVCache, kind: int, tok: int, pos: int, taps: bool = False) -> TokenOut:
    """Feed one token; it attends to every token already in `kv` and to itself."""
    m, w = model, model.w
    x = m.embed(kind, tok, pos)
    attn_taps = [] if taps else None
    for l in range(m.L):
        p = f"l{l}."
        a = m.R(m.layer_norm(x, w[p + "ln1_g"], w[p + "ln1_b"]))
        qkv = m.R(w[p + "wqkv"] @ a + w[p + "bqkv"])
        q = qkv[:m.d].reshape(m.H, m.dh)
        k = qkv[m.d:2 * m.d].reshape(m.H, m.dh)
        v = qkv[2 * m.d:].reshape(m.H, m.dh)
        kv.append(l, k, v)
        Km, Vm = kv.rows(l, kv.own + 1)                    # [t, H, dh], includes this token
        s = np.einsum("hd,thd->ht", q, Km) * m.scale        # [H, t]
        e = np.exp(s - s.max(axis=1, keepdims=True))
        o = np.einsum("ht,thd->hd", e, Vm) / e.sum(axis=1, keepdims=True)
        o = m.R(o).reshape(m.d)
        if taps:
            attn_taps.append(o.copy())
        x = x + w[p + "wo"] @ o + w[p + "bo"]
        a2 = m.R(m.layer_norm(x, w[p + "ln2_g"], w[p + "ln2_b"]))
        mid = m.R(np.maximum(w[p + "w1"] @ a2 + w[p + "b1"], 0.0))
        x = x + w[p + "w2"] @ mid + w[p + "b2"]
    kv.advance()
    h = m.R(m.layer_norm(x, w["lnf_g"], w["lnf_b"]))
    return TokenOut(h=h, logits=w["lm"] @ h, attn=attn_taps)


@dataclass
class TreeOut:
    h: np.ndarray             # [N, d]
    logits: np.ndarray        # [N, V]
    K: np.ndarray             # [L, N, H, dh]
    V: np.ndarray             # [L, N, H, dh]
    attn: List[np.ndarray]    # per layer [N, d]


def forward_tree(model: Model, kv: KVCache, kinds, toks, positions, mask: np.ndarray) -> TreeOut:
    """Score N new tokens in one pass (Sec. II-A, tree attention).

    Every new token attends to all tokens in `kv` and to the new tokens m with
    mask[n, m] true (its ancestors and itself).  `kv` is not modified."""
    m, w = model, model.w
    N = len(toks)
    x = np.stack([m.embed(int(kinds[i]), int(toks[i]), int(positions[i])) for i in range(N)])
    S = kv.n
    Ks = np.zeros((m.L, N, m.H, m.dh)); Vs = np.zeros_like(Ks)
    attn = []
    neg = np.where(mask, 0.0, -np.inf)                       # [N, N]
    for l in range(m.L):
        p = f"l{l}."
        a = m.R(m.layer_norm(x, w[p + "ln1_g"], w[p + "ln1_b"]))
        qkv = m.R(a @ w[p + "wqkv"].T + w[p + "bqkv"])
        q = qkv[:, :m.d].reshape(N, m.H, m.dh)
        k = qkv[:, m.d:2 * m.d].reshape(N, m.H, m.dh)
        v = qkv[:, 2 * m.d:].reshape(N, m.H, m.dh)
        Ks[l], Vs[l] = k, v
        Kc, Vc = kv.rows(l, kv.own)                          # [S, H, dh]
        s_ctx = np.einsum("nhd,thd->hnt", q, Kc) * m.scale   # [H, N, S]
        s_new = np.einsum("nhd,mhd->hnm", q, k) * m.scale + neg[None]
        s = np.concatenate([s_ctx, s_new], axis=2)
        e = np.exp(s - s.max(axis=2, keepdims=True))
        o = (np.einsum("hnt,thd->nhd", e[:, :, :S], Vc) + np.einsum("hnm,mhd->nhd", e[:, :, S:], v))
        o = o / e.sum(axis=2).T[:, :, None]
        o = m.R(o).reshape(N, m.d)
        attn.append(o.copy())
        x = x + o @ w[p + "wo"].T + w[p + "bo"]
        a2 = m.R(m.layer_norm(x, w[p + "ln2_g"], w[p + "ln2_b"]))
        mid = m.R(np.maximum(a2 @ w[p + "w1"].T + w[p + "b1"], 0.0))
        x = x + mid @ w[p + "w2"].T + w[p + "b2"]
    h = m.R(m.layer_norm(x, w["lnf_g"], w["lnf_b"]))
    return TreeOut(h=h, logits=h @ w["lm"].T, K=Ks, V=Vs, attn=attn)


def draft_logits(model: Model, h: np.ndarray) -> np.ndarray:
    """Logits of the draft heads at hidden state h: [n_draft, V].

    Head i (i = 1..n_draft) predicts the (i+1)-th next token (Sec. II-A); each is
    z = h + SiLU(W h + b) followed by its own vocabulary projection."""
    m, w = model, model.w
    out = np.zeros((m.n_draft, m.V))
    for i in range(m.n_draft):
        t = w[f"draft{i}.w"] @ h + w[f"draft{i}.b"]
        z = m.R(h + t / (1.0 + np.exp(-t)))
        out[i] = w[f"draft{i}.u"] @ z
    return out
