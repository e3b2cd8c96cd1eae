"""Sampling side of the oracle (test infrastructure only).

Algorithm 1 draws, at every position of a branch, tau samples from the
nucleus of the base head's distribution; a candidate is accepted when it is one
of them (Sec. II-C).  The draws are read here as sampling *without*
replacement, realised with the Gumbel-top-tau construction: perturb every
log-probability with independent Gumbel noise and keep the tau largest.  The
first of them is distributed as one ordinary multinomial draw, so tau = 1 is
ordinary sampling.

Noise is a pure function of (seed, sequence, absolute position of the token
being predicted, token id), so the sample for a position does not depend on how
the position was reached (by which tree, or by plain one-token decoding).

Integers are decided on float32 keys, ties broken towards the lower token id.
"""
from __future__ import annotations

import numpy as np

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15


def _mix_int(z: int) -> int:
    """Output function of the splitmix64 generator (Steele, Lea, Flood 2014)."""
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _mix_arr(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def uniform23(seed: int, seq: int, pos: int, n_tokens: int) -> np.ndarray:
    """u[token] in (0,1): 23 hashed bits x, u = (x + 1/2) / 2^23, exact in float32."""
    a = _mix_int(seed + _GOLDEN * (seq + 1))
    b = _mix_int(a + _GOLDEN * (pos + 1))
    tok = np.arange(1, n_tokens + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        c = _mix_arr(np.uint64(b) + np.uint64(_GOLDEN) * tok)
    x = (c >> np.uint64(41)).astype(np.float64)
    return ((x + 0.5) / float(1 << 23)).astype(np.float32)


def gumbel_noise(seed: int, seq: int, pos: int, n_tokens: int) -> np.ndarray:
    u = uniform23(seed, seq, pos, n_tokens).astype(np.float64)
    return (-np.log(-np.log(u))).astype(np.float32)


def masked_logits32(logits, eos_id: int, eos_masked: bool) -> np.ndarray:
    l = np.asarray(logits, dtype=np.float64).astype(np.float32)
    if eos_masked:
        l[eos_id] = -np.inf
    return l


def decision_keys(logits32: np.ndarray, temperature: float, seed: int, seq: int, pos: int,
                  noise: bool = True) -> np.ndarray:
    """float32 keys whose descending order is the order in which tokens are drawn.

    temperature 0 (greedy) or noise=False: the logits themselves."""
    if temperature == 0.0 or not noise:
        return logits32.copy()
    inv_t = np.float32(1.0 / float(temperature))
    g = gumbel_noise(seed, seq, pos, logits32.shape[0])
    return (logits32 * inv_t).astype(np.float32) + g


def _probs(logits32: np.ndarray, temperature: float) -> np.ndarray:
    z = logits32.astype(np.float64) / float(temperature)
    e = np.exp(z - z.max())
    return e / e.sum()


def _order(values: np.ndarray) -> np.ndarray:
    """Token ids sorted by value descending, then id ascending."""
    ids = np.arange(values.shape[0])
    return np.lexsort((ids, -values.astype(np.float64)))


def nucleus_sorted(logits32: np.ndarray, temperature: float, top_p: float) -> np.ndarray:
    """Boolean membership of the top-p nucleus, by the sort-and-accumulate definition:
    the shortest prefix, in descending probability, whose mass reaches top_p
    (the token that crosses the threshold is in).  Tokens of probability zero are
    never in.  Greedy decoding and top_p >= 1 switch the nucleus off."""
    finite = np.isfinite(logits32)
    if temperature == 0.0 or top_p >= 1.0:
        return finite
    p = _probs(logits32, temperature)
    order = _order(p)
    before = np.concatenate([[0.0], np.cumsum(p[order])[:-1]])
    member = np.zeros(p.shape[0], dtype=bool)
    member[order] = before < top_p
    return member & finite


def nucleus_mass_before(logits32: np.ndarray, temperature: float, c: int) -> float:
    """Probability mass of the tokens that precede c in descending-probability order."""
    p = _probs(logits32, temperature)
    ids = np.arange(p.shape[0])
    ahead = (p > p[c]) | ((p == p[c]) & (ids < c))
    return float(p[ahead].sum())


def sample_set(keys: np.ndarray, nucleus: np.ndarray, tau: int) -> list:
    """The tau draws v (Alg. 1, line 3), in the order drawn: the members of the
    nucleus sorted by key (descending, lower id first among equals), cut at tau."""
    order = [int(j) for j in _order(keys) if nucleus[j]]
    return order[:tau]


def root_token(keys: np.ndarray, nucleus: np.ndarray) -> int:
    """The base head's ordinary single sample = the first draw."""
    return sample_set(keys, nucleus, 1)[0]


def in_set_by_rank_count(keys: np.ndarray, nucleus: np.ndarray, tau: int, c: int) -> bool:
    """Same membership as `c in sample_set(...)`, without sorting: c is in the
    nucleus and fewer than tau nucleus members precede it in key order."""
    if not nucleus[c]:
        return False
    ids = np.arange(keys.shape[0])
    ahead = nucleus & ((keys > keys[c]) | ((keys == keys[c]) & (ids < c)))
    return int(ahead.sum()) < tau


def topk_ids(logits32: np.ndarray, k: int) -> np.ndarray:
    """Ids of the k largest logits, descending, lower id first among equals."""
    return _order(logits32)[:k].astype(np.int32)
