"""CPU oracle for the VADUSA tree draft-and-verify step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the paper's decoding
procedure computes (Sec. II-A: draft heads and candidate tree; Sec. II-C and
Algorithm 1: verification with the tolerance mechanism and the choice of the
longest, then leftmost, accepted branch; Sec. II-D: greedy sparse-tree
construction), on a plain pre-LN decoder-only transformer.  Floating point is float64 throughout; in "bf16" models the values
the model *stores* in bf16 are rounded at the stated points; the keys that
decide integers are formed in float32.

Nothing here is used by the product path.  Only the tests, the smoke check and
the benchmark's CPU-baseline leg import this package; it imports nothing from
the CUDA package, and shares no code with it.

Parity unpinned (nothing in the paper fixes them): the value of top-p, the
synthetic tree template, and the architecture details the paper delegates to
VALL-E (pre-LN, learned positions, ReLU feed-forward, bias placement).
"""
from .numerics import round_bf16
from .model import Model, KVCache, forward_token, forward_tree, draft_logits
from .sampling import (uniform23, gumbel_noise, decision_keys, nucleus_sorted, sample_set,
                       root_token, in_set_by_rank_count, topk_ids, nucleus_mass_before)
from .verify import verify_branch, select_best, accept_from_edges, tree_edge_accepts
from .decode import (Sampling, ar_decode, prefill, prefill_blocked, State, vadusa_iteration,
                     vadusa_generate, build_tree_tokens, IterationTrace, sample_next, draws_at,
                     draft_topk)
from .tree_build import (greedy_tree, best_tree_brute_force, expected_length, path_probability)
from . import tree_build

__all__ = [n for n in dir() if not n.startswith("_")]
