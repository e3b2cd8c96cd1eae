"""Model shapes and the five synthetic workloads (shapes only, no arithmetic).

The workloads stand in for the paper's evaluation sets, which are not
available: they keep its shapes (12 layers, 16 heads, d 1024, FFN 4096 in
Sec. III-A.1; 4 draft heads, 64-node sparse tree, top-k 10 and tolerance 1..4
in Sec. III-A.3; 50-75 Hz token streams of about ten seconds in Sec. I).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int                 # codec ids + one EOS id (the last id)
    n_draft_heads: int
    dtype: str                 # "fp32" or "bf16" (storage type of matrices, KV and activations)
    n_phonemes: int = 64
    max_pos: int = 8192
    ln_eps: float = 1e-5

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    @property
    def eos_id(self) -> int:
        return self.vocab - 1


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                         # 1..5, used in seeds (seed = 1000*index + item)
    shape: ModelShape
    batch: int
    tree_nodes: int
    tree_caps: Tuple[int, ...]         # usable top-k ranks per draft depth
    tau: int                           # tolerance
    temperature: float                 # 0 means greedy
    top_p: float = 1.0
    eos_masked: bool = True
    gen_tokens: int = 0                # tokens to generate per sequence (0: iteration-bounded)
    iterations: int = 0                # speculative iterations per sequence (0: token-bounded)
    phoneme_len: Tuple[int, int] = (0, 0)   # inclusive range
    prompt_len: int = 0
    context_len: Tuple[int, int] = (0, 0)   # inclusive range of pre-existing KV lengths (C4, C5)
    kv_block: int = 64
    random_topology: bool = False      # C5: per-sequence random trees
    topology_max_depth: int = 5
    tau_sweep: Tuple[int, ...] = field(default_factory=tuple)

    def seed(self, item: int = 0) -> int:
        return 1000 * self.index + item


_TINY = ModelShape(n_layers=2, d_model=256, n_heads=4, d_ffn=1024, vocab=1025,
                   n_draft_heads=3, dtype="fp32")
_VALLE_1025 = ModelShape(n_layers=12, d_model=1024, n_heads=16, d_ffn=4096, vocab=1025,
                         n_draft_heads=4, dtype="bf16")
_VALLE_2049 = replace(_VALLE_1025, vocab=2049)

WORKLOADS = {
    "C1": Workload(name="C1", index=1, shape=_TINY, batch=1, tree_nodes=16, tree_caps=(10, 5, 3),
                   tau=1, temperature=0.0, gen_tokens=100, phoneme_len=(32, 32), prompt_len=75),
    "C2": Workload(name="C2", index=2, shape=_VALLE_1025, batch=1, tree_nodes=64,
                   tree_caps=(10, 5, 3, 2), tau=3, temperature=1.0, gen_tokens=750,
                   phoneme_len=(100, 100), prompt_len=225),
    "C3": Workload(name="C3", index=3, shape=_VALLE_2049, batch=16, tree_nodes=42,
                   tree_caps=(10, 5, 3, 2), tau=5, temperature=0.8, gen_tokens=500,
                   phoneme_len=(40, 120), prompt_len=150),
    "C4": Workload(name="C4", index=4, shape=_VALLE_1025, batch=32, tree_nodes=64,
                   tree_caps=(10, 5, 3, 2), tau=3, temperature=1.0, iterations=256,
                   phoneme_len=(100, 100), context_len=(1000, 4000), tau_sweep=(1, 3, 5)),
    "C5": Workload(name="C5", index=5, shape=_VALLE_1025, batch=64, tree_nodes=64,
                   tree_caps=(10, 5, 3, 2), tau=3, temperature=1.0, iterations=1,
                   context_len=(256, 3000), random_topology=True),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


def toy_workload(dtype: str = "fp32", n_layers: int = 2, d_model: int = 64, n_heads: int = 2,
                 d_ffn: int = 128, vocab: int = 41, n_draft_heads: int = 3, tree_nodes: int = 10,
                 tree_caps: Tuple[int, ...] = (4, 3, 2), tau: int = 2, temperature: float = 1.0,
                 batch: int = 1, index: int = 9, max_pos: int = 512, n_phonemes: int = 8,
                 gen_tokens: int = 12, phoneme_len=(5, 5), prompt_len: int = 7) -> Workload:
    """A very small model for brute-force and unit tests."""
    shape = ModelShape(n_layers=n_layers, d_model=d_model, n_heads=n_heads, d_ffn=d_ffn, vocab=vocab,
                       n_draft_heads=n_draft_heads, dtype=dtype, n_phonemes=n_phonemes, max_pos=max_pos)
    return Workload(name="toy", index=index, shape=shape, batch=batch, tree_nodes=tree_nodes,
                    tree_caps=tree_caps, tau=tau, temperature=temperature, gen_tokens=gen_tokens,
                    phoneme_len=phoneme_len, prompt_len=prompt_len)
