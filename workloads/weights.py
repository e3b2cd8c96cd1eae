"""Random-init weights (seeded normal, std 0.02) for the decoder-only speech-token model.

Every tensor is drawn from its own Philox stream keyed by (seed, tensor name), so
the values do not depend on the order of generation.  In "bf16" shapes the
matrices and embedding tables are rounded once to bf16-representable values
(round to nearest even) and returned as float32; vectors (biases, LayerNorm
parameters) stay float32.  This is input preparation only.
"""
from __future__ import annotations

import zlib
from typing import Dict

import numpy as np

from .configs import ModelShape


def round_to_bf16_values(a: np.ndarray) -> np.ndarray:
    """float32 array whose values are the nearest-even bf16 neighbours of `a`."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).reshape(a.shape)


def _stream(seed: int, name: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), zlib.crc32(name.encode())]))


def _normal(seed: int, name: str, shape, std: float = 0.02, mean: float = 0.0) -> np.ndarray:
    g = _stream(seed, name)
    return (mean + std * g.standard_normal(size=shape, dtype=np.float32)).astype(np.float32)


def make_weights(shape: ModelShape, seed: int) -> Dict[str, np.ndarray]:
    """Dictionary of float32 arrays; matrices are [out_features, in_features]."""
    d, f, v, hd = shape.d_model, shape.d_ffn, shape.vocab, shape.n_draft_heads
    w: Dict[str, np.ndarray] = {}

    def mat(name, *dims):
        a = _normal(seed, name, dims)
        w[name] = round_to_bf16_values(a) if shape.dtype == "bf16" else a

    def vec(name, n, mean=0.0):
        w[name] = _normal(seed, name, (n,), mean=mean)

    mat("emb_audio", v, d)
    mat("emb_phon", shape.n_phonemes, d)
    mat("pos", shape.max_pos, d)
    for l in range(shape.n_layers):
        p = f"l{l}."
        vec(p + "ln1_g", d, mean=1.0); vec(p + "ln1_b", d)
        mat(p + "wqkv", 3 * d, d);     vec(p + "bqkv", 3 * d)
        mat(p + "wo", d, d);           vec(p + "bo", d)
        vec(p + "ln2_g", d, mean=1.0); vec(p + "ln2_b", d)
        mat(p + "w1", f, d);           vec(p + "b1", f)
        mat(p + "w2", d, f);           vec(p + "b2", d)
    vec("lnf_g", d, mean=1.0); vec("lnf_b", d)
    mat("lm", v, d)
    for i in range(hd):
        p = f"draft{i}."
        mat(p + "w", d, d); vec(p + "b", d)
        mat(p + "u", v, d)
    return w
