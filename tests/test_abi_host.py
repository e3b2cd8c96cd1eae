"""Host-side checks of the C ABI that need no GPU: the library builds, loads and
exports every symbol the header declares; sizing and layout calls; validation."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import workloads as W
import paper_2410_21951_b200 as P
from paper_2410_21951_b200.binding import EXPORTS, Config, TensorInfo, Weights, make_config

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "vadusa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vadusa_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = P.lib()
    syms = declared_symbols()
    assert len(syms) >= 18
    for s in syms:
        assert hasattr(L, s), s
    assert sorted(EXPORTS) == syms


def test_sizes_and_weight_layout():
    L = P.lib()
    for name in ("C1", "C2", "C3"):
        wl = W.workload(name)
        cfg = make_config(wl.shape, wl.batch, wl.tree_nodes, 20, 40)
        assert C.sizeof(Config) == cfg.struct_size
        infos = P.tensor_infos(cfg)
        names = [t.name.decode() for t in infos]
        assert len(set(names)) == len(names)
        assert names[:3] == ["emb_audio", "emb_phon", "pos"]
        end = 0
        es = 2 if wl.shape.dtype == "bf16" else 4
        for t in infos:
            assert t.offset % 256 == 0 and t.offset >= end
            assert t.nbytes == t.rows_padded * t.cols * (es if t.is_matrix else 4)
            end = t.offset + t.nbytes
        assert L.vadusa_weights_bytes(C.byref(cfg)) >= end
        lm = infos[names.index("lm")]
        assert lm.rows == wl.shape.vocab and lm.rows_padded % 128 == 0 and lm.rows_padded >= lm.rows
        # draft matrices are evenly spaced (batched product over heads)
        offs = [infos[names.index(f"draft{i}.u")].offset for i in range(wl.shape.n_draft_heads)]
        assert len(set(np.diff(offs))) == 1
        sh = wl.shape
        assert L.vadusa_kv_pool_bytes(C.byref(cfg)) == sh.n_layers * 40 * 2 * sh.d_model * 64 * es
        assert L.vadusa_workspace_bytes(C.byref(cfg)) > wl.batch * wl.tree_nodes * sh.d_ffn * es


def test_pack_weights_round_trip():
    wl = W.toy_workload(dtype="bf16")
    w = W.make_weights(wl.shape, 1)
    cfg = make_config(wl.shape, 1, 16, 4, 8)
    blob = P.pack_weights(cfg, w)
    for t in P.tensor_infos(cfg):
        name = t.name.decode()
        raw = blob[t.offset:t.offset + t.nbytes]
        if t.is_matrix:
            bits = raw.view(np.uint16).astype(np.uint32) << 16
            got = bits.view(np.float32).reshape(t.rows_padded, t.cols)
            assert np.array_equal(got[:t.rows], w[name]) and not got[t.rows:].any()
        else:
            assert np.array_equal(raw.view(np.float32), w[name])
    bad = dict(w); bad["lm"] = w["lm"] + np.float32(1e-3)
    with pytest.raises(ValueError):
        P.pack_weights(cfg, bad)


@pytest.mark.parametrize("field,value", [("d_model", 100), ("n_heads", 3), ("kv_block", 32), ("dtype", 2),
                                          ("max_tree_nodes", 129), ("prefill_rows", -1), ("draft_topk", 0), ("n_draft_heads", 16),
                                          ("struct_size", 8), ("abi_version", 99), ("kv_num_blocks", 0)])
def test_bad_configurations_are_rejected(field, value):
    L = P.lib()
    cfg = make_config(W.workload("C1").shape, 1, 16, 8, 8)
    setattr(cfg, field, value)
    assert L.vadusa_workspace_bytes(C.byref(cfg)) < 0
    assert L.vadusa_weight_count(C.byref(cfg)) < 0
    t = TensorInfo()
    assert L.vadusa_weight_info(C.byref(cfg), 0, C.byref(t)) == 1


def test_init_reports_errors_without_touching_a_gpu():
    L = P.lib()
    cfg = make_config(W.workload("C1").shape, 1, 16, 8, 8)
    ctx = C.c_void_p()
    w = Weights(None, 0)
    assert L.vadusa_init(C.byref(w), C.byref(cfg), C.byref(ctx)) == 1      # EINVAL: no weights
    assert b"weights" in L.vadusa_last_error(ctx)
    L.vadusa_destroy(ctx)
    buf = np.zeros(1024, dtype=np.uint8)
    w = Weights(buf.ctypes.data, buf.nbytes)
    assert L.vadusa_init(C.byref(w), C.byref(cfg), C.byref(ctx)) == 2      # ENOMEM: blob too small
    L.vadusa_destroy(ctx)
    assert L.vadusa_init(C.byref(w), C.byref(cfg), None) == 1
    assert L.vadusa_destroy(None) == 1
    assert L.vadusa_check(None) == 1


def test_python_binding_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    wl = W.toy_workload()
    with pytest.raises(P.VadusaError):
        P.Vadusa(wl.shape, W.make_weights(wl.shape, 1), 1, 16, 4, 8)
