"""Block tables for a paged KV cache: pages are handed out from a shuffled free
list so that the tables are non-contiguous, as in a serving system."""
from __future__ import annotations

import numpy as np


def shuffled_block_table(tokens_per_seq, kv_block: int, seed: int, spare_pages: int = 0):
    """Returns (block_table int32 [B, max_pages], n_pages_total).

    Sequence b owns ceil(tokens_per_seq[b] / kv_block) distinct pages; unused
    entries are -1.  `spare_pages` extra pages exist in the pool but belong to
    no sequence."""
    need = [(int(t) + kv_block - 1) // kv_block for t in tokens_per_seq]
    total = sum(need) + spare_pages
    g = np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), 5]))
    free = g.permutation(total).astype(np.int32)
    table = np.full((len(need), max(need) if need else 0), -1, dtype=np.int32)
    k = 0
    for b, n in enumerate(need):
        table[b, :n] = free[k:k + n]
        k += n
    return table, total
