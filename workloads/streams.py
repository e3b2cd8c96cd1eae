"""Seeded token streams shaped like VALL-E inputs: a phoneme prefix and an
acoustic prompt whose codec ids repeat from frame to frame (order-1 Markov
chain with self-transition probability 0.3, as 50-75 Hz codec streams do)."""
from __future__ import annotations

from typing import List, Tuple

import numpy as np

from .configs import Workload


def _gen(seed: int, tag: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), tag]))


def phonemes(n: int, n_ids: int, seed: int) -> np.ndarray:
    return _gen(seed, 1).integers(0, n_ids, size=n, dtype=np.int64).astype(np.int32)


def markov_prompt(n: int, n_ids: int, seed: int, p_stay: float = 0.3) -> np.ndarray:
    """x0 uniform; then stay with probability p_stay, else uniform over the other ids."""
    g = _gen(seed, 2)
    out = np.empty(n, dtype=np.int32)
    if n == 0:
        return out
    stay = g.random(size=n) < p_stay
    jump = g.integers(0, n_ids - 1, size=n, dtype=np.int64)
    cur = int(g.integers(0, n_ids))
    out[0] = cur
    for t in range(1, n):
        if not stay[t]:
            j = int(jump[t])
            cur = j if j < cur else j + 1          # uniform over ids other than cur
        out[t] = cur
    return out


def ragged_lengths(n: int, lo: int, hi: int, seed: int) -> np.ndarray:
    """n lengths uniform in [lo, hi] inclusive."""
    return _gen(seed, 3).integers(lo, hi + 1, size=n, dtype=np.int64).astype(np.int32)


def prefix_for(wl: Workload, item: int) -> Tuple[np.ndarray, np.ndarray]:
    """(phoneme ids, prompt codec ids) of sequence `item` of a workload."""
    seed = wl.seed(item)
    n_codec = wl.shape.vocab - 1
    if wl.context_len != (0, 0):
        total = int(ragged_lengths(wl.batch, wl.context_len[0], wl.context_len[1], wl.seed(900))[item])
        n_ph = min(wl.phoneme_len[0], total)
        return phonemes(n_ph, wl.shape.n_phonemes, seed), markov_prompt(total - n_ph, n_codec, seed)
    lo, hi = wl.phoneme_len
    n_ph = lo if lo == hi else int(ragged_lengths(wl.batch, lo, hi, wl.seed(901))[item])
    return phonemes(n_ph, wl.shape.n_phonemes, seed), markov_prompt(wl.prompt_len, n_codec, seed)
