"""Fitting of the draft heads with the base model frozen (test infrastructure only).

Paper Sec. II-A: the i-th draft head (i >= 1) predicts the (i+1)-th next token under a
cross-entropy loss multiplied by lambda^i, lambda in (0, 1); Sec. III-A.2: the heads are trained
with the base model fixed ("wot"), lambda = 0.8, learning rate 0.002, 40 warm-up steps.  A head is
z = h + SiLU(W h + b), logits = U z (Sec. III-A.1).

Everything here is float64 and written out step by step: forward, loss, the gradient of every
parameter by the chain rule, and the update.  Readings (the paper names no optimiser and no
normalisation of the loss): each head's cross-entropy is averaged over the positions that have
a target; the optimiser is Adam (beta1 0.9, beta2 0.999, eps 1e-8, no weight decay) with the
learning rate rising linearly over the warm-up steps.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Tuple

import numpy as np


def silu(x):
    return x / (1.0 + np.exp(-x))


def silu_grad(x):
    s = 1.0 / (1.0 + np.exp(-x))
    return s * (1.0 + x * (1.0 - s))


def heads_loss(W, b, U, h, targets, lam: float) -> Tuple[float, np.ndarray]:
    """Loss of all heads on hidden states h [T, d] with targets [T, heads] (-1: no target).
    W [heads, d, d], b [heads, d], U [heads, V, d].  Returns (total, per-head mean cross-entropies)."""
    n_heads = W.shape[0]
    per = np.zeros(n_heads)
    total = 0.0
    for i in range(n_heads):
        z = h + silu(h @ W[i].T + b[i])
        logits = z @ U[i].T
        valid = targets[:, i] >= 0
        if not np.any(valid):
            continue
        lg = logits[valid]
        lse = lg.max(axis=1) + np.log(np.exp(lg - lg.max(axis=1, keepdims=True)).sum(axis=1))
        ce = lse - lg[np.arange(lg.shape[0]), targets[valid, i]]
        per[i] = ce.mean()
        total += lam ** (i + 1) * per[i]
    return total, per


def heads_grads(W, b, U, h, targets, lam: float):
    """(loss, per-head cross-entropies, dW, db, dU) of `heads_loss`."""
    n_heads = W.shape[0]
    dW, db, dU = np.zeros_like(W), np.zeros_like(b), np.zeros_like(U)
    per = np.zeros(n_heads)
    total = 0.0
    for i in range(n_heads):
        pre = h @ W[i].T + b[i]
        z = h + silu(pre)
        logits = z @ U[i].T
        valid = targets[:, i] >= 0
        n = int(valid.sum())
        if n == 0:
            continue
        mx = logits.max(axis=1, keepdims=True)
        p = np.exp(logits - mx)
        p /= p.sum(axis=1, keepdims=True)
        rows = np.nonzero(valid)[0]
        per[i] = float(np.mean(-np.log(p[rows, targets[rows, i]])))
        total += lam ** (i + 1) * per[i]
        dl = p.copy()
        dl[rows, targets[rows, i]] -= 1.0
        dl[~valid] = 0.0
        dl *= lam ** (i + 1) / n                      # d loss / d logits
        dU[i] = dl.T @ z
        dz = dl @ U[i]
        dpre = dz * silu_grad(pre)
        dW[i] = dpre.T @ h
        db[i] = dpre.sum(axis=0)
    return total, per, dW, db, dU


@dataclass
class AdamState:
    m: np.ndarray
    v: np.ndarray


def adam_update(param, grad, st: AdamState, step: int, lr: float, beta1=0.9, beta2=0.999, eps=1e-8):
    """One Adam step (step counts from 1); returns the new parameter."""
    st.m = beta1 * st.m + (1.0 - beta1) * grad
    st.v = beta2 * st.v + (1.0 - beta2) * grad * grad
    mh = st.m / (1.0 - beta1 ** step)
    vh = st.v / (1.0 - beta2 ** step)
    return param - lr * mh / (np.sqrt(vh) + eps)


def warmup_lr(step: int, lr: float, warmup: int) -> float:
    """Learning rate of step `step` (from 1): linear rise over `warmup` steps, then constant."""
    return lr * min(1.0, step / float(max(warmup, 1)))


class HeadFitter:
    """Holds float64 copies of the heads and their Adam moments; `step` does one update."""

    def __init__(self, W, b, U, lam: float = 0.8, lr: float = 0.002, warmup: int = 40):
        self.W, self.b, self.U = (np.array(a, dtype=np.float64) for a in (W, b, U))
        self.lam, self.lr, self.warmup = lam, lr, warmup
        self.t = 0
        self.st = [AdamState(np.zeros_like(a), np.zeros_like(a)) for a in (self.W, self.b, self.U)]

    def step(self, h, targets):
        loss, per, dW, db, dU = heads_grads(self.W, self.b, self.U, np.asarray(h, dtype=np.float64), targets, self.lam)
        self.t += 1
        lr = warmup_lr(self.t, self.lr, self.warmup)
        self.W = adam_update(self.W, dW, self.st[0], self.t, lr)
        self.b = adam_update(self.b, db, self.st[1], self.t, lr)
        self.U = adam_update(self.U, dU, self.st[2], self.t, lr)
        return loss, per
