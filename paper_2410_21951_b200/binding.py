"""ctypes binding of libvadusa (argument marshalling only).

Function names and arguments follow include/vadusa.h.  PyTorch is used for
device memory and the stream, nothing else.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import build as _build

MAX_PATH = 16          # VADUSA_MAX_DEPTH + 1
ABI_VERSION = 2

STATUS = {0: "OK", 1: "EINVAL", 2: "ENOMEM", 3: "ECUDA", 4: "ECAPACITY", 5: "ESTATE", 6: "ETIMEOUT"}


class VadusaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"libvadusa: {STATUS.get(status, status)}: {message}")
        self.status = status


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("abi_version", C.c_uint32),
                ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab", C.c_int32), ("n_phonemes", C.c_int32), ("max_pos", C.c_int32), ("dtype", C.c_int32),
                ("n_draft_heads", C.c_int32), ("draft_topk", C.c_int32), ("max_batch", C.c_int32),
                ("max_tree_nodes", C.c_int32), ("kv_block", C.c_int32), ("max_blocks_per_seq", C.c_int32),
                ("prefill_rows", C.c_int32), ("reserved0", C.c_int32),
                ("kv_num_blocks", C.c_int64), ("ln_eps", C.c_float), ("device", C.c_int32),
                ("kv_pool", C.c_void_p), ("kv_pool_bytes", C.c_int64),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_int64), ("stream", C.c_void_p)]


class Weights(C.Structure):
    _fields_ = [("blob", C.c_void_p), ("nbytes", C.c_int64)]


class TensorInfo(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("offset", C.c_int64), ("nbytes", C.c_int64), ("rows", C.c_int32),
                ("cols", C.c_int32), ("rows_padded", C.c_int32), ("is_matrix", C.c_int32)]


class Sampling(C.Structure):
    _fields_ = [("tau", C.c_int32), ("temperature", C.c_float), ("top_p", C.c_float), ("eos_masked", C.c_int32),
                ("accept_rule", C.c_int32), ("seed", C.c_uint64)]

    @classmethod
    def make(cls, tau=1, temperature=0.0, top_p=1.0, eos_masked=True, accept_rule=0, seed=0):
        return cls(int(tau), float(temperature), float(top_p), int(bool(eos_masked)), int(accept_rule), int(seed))


class Stats(C.Structure):
    _fields_ = [("iterations", C.c_int64), ("tokens_generated", C.c_int64), ("elapsed_ms", C.c_double),
                ("kernel_launches", C.c_int64)]


class KernelTime(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_int64), ("total_ms", C.c_double)]


EXPORTS = ["vadusa_workspace_bytes", "vadusa_weights_bytes", "vadusa_kv_pool_bytes", "vadusa_weight_count",
           "vadusa_weight_info", "vadusa_init", "vadusa_destroy", "vadusa_last_error", "vadusa_set_tree",
           "vadusa_begin", "vadusa_prefill", "vadusa_load_state", "vadusa_draft", "vadusa_verify_step",
           "vadusa_accept_and_commit", "vadusa_generate", "vadusa_generate_host", "vadusa_get_lengths",
           "vadusa_check", "vadusa_kernel_launches", "vadusa_profile_begin", "vadusa_profile_end",
           "vadusa_accept_stats", "vadusa_build_sparse_tree", "vadusa_set_logit_bias", "vadusa_set_fused_pass", "vadusa_fused_pass_clusters", "vadusa_set_attention_stream",
           "vadusa_fit_state_bytes", "vadusa_fit_begin", "vadusa_fit_step", "vadusa_fit_end", "vadusa_set_prefill_tap",
           "vadusa_draft_topk_static", "vadusa_static_scratch_bytes", "vadusa_static_last_error"]

_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads libvadusa.so, building it first if its sources changed.  Raises if it
    cannot be built or loaded: there is no fallback."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    lib_ = C.CDLL(path or _build.build())
    P, I32, I64 = C.c_void_p, C.c_int32, C.c_int64
    cfgp = C.POINTER(Config)
    sig = {
        "vadusa_workspace_bytes": (I64, [cfgp]), "vadusa_weights_bytes": (I64, [cfgp]),
        "vadusa_kv_pool_bytes": (I64, [cfgp]), "vadusa_weight_count": (I32, [cfgp]),
        "vadusa_weight_info": (I32, [cfgp, I32, C.POINTER(TensorInfo)]),
        "vadusa_init": (I32, [C.POINTER(Weights), cfgp, C.POINTER(P)]),
        "vadusa_destroy": (I32, [P]), "vadusa_last_error": (C.c_char_p, [P]),
        "vadusa_set_tree": (I32, [P, I32, P, P, I32]),
        "vadusa_begin": (I32, [P, I32, P, P]),
        "vadusa_prefill": (I32, [P, P, P, I32]),
        "vadusa_load_state": (I32, [P, P, P]),
        "vadusa_draft": (I32, [P, C.POINTER(Sampling), P, P]),
        "vadusa_verify_step": (I32, [P, P, P, P, P]),
        "vadusa_accept_and_commit": (I32, [P, C.POINTER(Sampling), P, P, P, P, P, P, P]),
        "vadusa_generate": (I32, [P, C.POINTER(Sampling), I32, I32, P, P, C.POINTER(Stats)]),
        "vadusa_generate_host": (I32, [P, C.POINTER(Sampling), I32, P, P, P, I32, I32, P, P, C.POINTER(Stats)]),
        "vadusa_get_lengths": (I32, [P, P]), "vadusa_check": (I32, [P]),
        "vadusa_kernel_launches": (I64, [P]),
        "vadusa_set_fused_pass": (I32, [P, I32]),
        "vadusa_set_attention_stream": (I32, [P, I32]),
        "vadusa_fused_pass_clusters": (I32, [P]),
        "vadusa_fit_state_bytes": (I64, [cfgp, I32]),
        "vadusa_fit_begin": (I32, [P, P, I64, I32, C.c_float, C.c_float, I32]),
        "vadusa_fit_step": (I32, [P, P, P, I32, P]),
        "vadusa_fit_end": (I32, [P]),
        "vadusa_set_prefill_tap": (I32, [P, P, I32]),
        "vadusa_draft_topk_static": (I32, [P, P, P, P, I32, I32, I32, I32, I32, I32, I32, P, P]),
        "vadusa_static_scratch_bytes": (I64, []),
        "vadusa_static_last_error": (C.c_char_p, []),
        "vadusa_accept_stats": (I32, [P, P, P, I32]),
        "vadusa_set_logit_bias": (I32, [P, P, I32]),
        "vadusa_build_sparse_tree": (I32, [P, I32, I32, I32, P, P, P]),
        "vadusa_profile_begin": (I32, [P]),
        "vadusa_profile_end": (I32, [P, C.POINTER(KernelTime), I32, C.POINTER(I32)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib_, name)
        fn.restype, fn.argtypes = res, args
    if path is None:
        _lib = lib_
    return lib_


def lib() -> C.CDLL:
    return load_library()


def make_config(shape, max_batch: int, max_tree_nodes: int, max_blocks_per_seq: int, kv_num_blocks: int,
                draft_topk: int = 10, device: int = 0, prefill_rows: int = 0) -> Config:
    """Config from a model shape (any object with the fields of workloads.ModelShape)."""
    c = Config()
    c.struct_size, c.abi_version = C.sizeof(Config), ABI_VERSION
    c.n_layers, c.d_model, c.n_heads, c.d_ffn = shape.n_layers, shape.d_model, shape.n_heads, shape.d_ffn
    c.vocab, c.n_phonemes, c.max_pos = shape.vocab, shape.n_phonemes, shape.max_pos
    c.dtype = 1 if shape.dtype == "bf16" else 0
    c.n_draft_heads, c.draft_topk = shape.n_draft_heads, min(draft_topk, shape.vocab - 1)
    c.max_batch, c.max_tree_nodes, c.kv_block = max_batch, max_tree_nodes, 64
    c.max_blocks_per_seq, c.kv_num_blocks = max_blocks_per_seq, kv_num_blocks
    c.ln_eps, c.device = shape.ln_eps, device
    c.prefill_rows, c.reserved0 = prefill_rows, 0
    return c


def tensor_infos(cfg: Config) -> List[TensorInfo]:
    L = lib()
    n = L.vadusa_weight_count(C.byref(cfg))
    if n < 0:
        raise VadusaError(1, "bad configuration")
    out = []
    for i in range(n):
        t = TensorInfo()
        st = L.vadusa_weight_info(C.byref(cfg), i, C.byref(t))
        if st:
            raise VadusaError(st, "vadusa_weight_info")
        out.append(t)
    return out


def _bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are exactly representable in bf16."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    if np.any(bits & 0xFFFF):
        raise ValueError("matrix values are not bf16-representable")
    return (bits >> 16).astype(np.uint16)


def pack_weights(cfg: Config, weights: Dict[str, np.ndarray]) -> np.ndarray:
    """The weight blob (host, uint8) in the layout vadusa_weight_info reports."""
    L = lib()
    total = L.vadusa_weights_bytes(C.byref(cfg))
    blob = np.zeros(total, dtype=np.uint8)
    for t in tensor_infos(cfg):
        name = t.name.decode()
        a = np.asarray(weights[name])
        if t.is_matrix:
            assert a.shape == (t.rows, t.cols), (name, a.shape, t.rows, t.cols)
            raw = (_bf16_bits(a) if cfg.dtype == 1 else np.ascontiguousarray(a, dtype=np.float32)).view(np.uint8)
        else:
            assert a.shape == (t.rows,), (name, a.shape)
            raw = np.ascontiguousarray(a, dtype=np.float32).view(np.uint8)
        raw = raw.reshape(-1)
        blob[t.offset:t.offset + raw.size] = raw
    return blob


def draft_topk_static(draft_w, draft_b, draft_u, hstar, dtype: int, batch: int, d_model: int, vocab: int,
                      n_draft_heads: int, topk: int, eos_masked: bool, topk_out, stream=None):
    """vadusa_draft_topk_static: device tensors in, device tensor out, no allocation in the library.
    `stream` is a torch stream (None: the legacy default stream)."""
    L = lib()
    st = L.vadusa_draft_topk_static(C.c_void_p(draft_w.data_ptr()), C.c_void_p(draft_b.data_ptr()),
                                    C.c_void_p(draft_u.data_ptr()), C.c_void_p(hstar.data_ptr()), dtype, batch,
                                    d_model, vocab, n_draft_heads, topk, int(bool(eos_masked)),
                                    C.c_void_p(topk_out.data_ptr()),
                                    C.c_void_p(stream.cuda_stream) if stream is not None else None)
    if st:
        raise VadusaError(st, L.vadusa_static_last_error().decode())


MAX_DEPTH, MAX_DRAFT_TOPK = 15, 16


def build_sparse_tree(prob: np.ndarray, n_nodes: int):
    """(parent, rank, expected accepted length) of the greedily grown tree; prob is [depth][topk].  Host only."""
    prob = np.ascontiguousarray(prob, dtype=np.float64)
    parent = np.zeros(n_nodes, dtype=np.int32)
    rank = np.zeros(n_nodes, dtype=np.int32)
    exp = C.c_double(0.0)
    st = lib().vadusa_build_sparse_tree(prob.ctypes.data, prob.shape[0], prob.shape[1], n_nodes, parent.ctypes.data,
                                        rank.ctypes.data, C.addressof(exp))
    if st:
        raise VadusaError(st, "vadusa_build_sparse_tree: bad arguments or fewer candidate nodes than asked for")
    return parent, rank, exp.value


class Vadusa:
    """One context of libvadusa together with the device buffers it works in."""

    def __init__(self, shape, weights: Dict[str, np.ndarray], max_batch: int, max_tree_nodes: int,
                 max_blocks_per_seq: int, kv_num_blocks: int, draft_topk: int = 10, device: int = 0,
                 stream=None, prefill_rows: int = 16):
        """prefill_rows: prefix chunks (of max_tree_nodes tokens) scored per prefill pass."""
        import torch
        self.torch = torch
        if not torch.cuda.is_available():
            raise VadusaError(3, "no CUDA device: this library has no CPU path")
        self.L = lib()
        self.shape = shape
        self.dev = torch.device("cuda", device)
        self.cfg = make_config(shape, max_batch, max_tree_nodes, max_blocks_per_seq, kv_num_blocks, draft_topk, device,
                               prefill_rows)
        self.tdtype = torch.bfloat16 if self.cfg.dtype == 1 else torch.float32
        self.blob = torch.from_numpy(pack_weights(self.cfg, weights)).to(self.dev)
        self.kv_pool = torch.zeros(self.L.vadusa_kv_pool_bytes(C.byref(self.cfg)), dtype=torch.uint8, device=self.dev)
        self.workspace = torch.zeros(self.L.vadusa_workspace_bytes(C.byref(self.cfg)), dtype=torch.uint8, device=self.dev)
        # a stream of its own: the legacy default stream cannot be captured into CUDA graphs
        self.stream = stream if stream is not None else torch.cuda.Stream(self.dev)
        self.cfg.kv_pool, self.cfg.kv_pool_bytes = self.kv_pool.data_ptr(), self.kv_pool.numel()
        self.cfg.workspace, self.cfg.workspace_bytes = self.workspace.data_ptr(), self.workspace.numel()
        self.cfg.stream = self.stream.cuda_stream
        self.ctx = C.c_void_p()
        w = Weights(self.blob.data_ptr(), self.blob.numel())
        st = self.L.vadusa_init(C.byref(w), C.byref(self.cfg), C.byref(self.ctx))
        if st:
            msg = self.L.vadusa_last_error(self.ctx).decode() if self.ctx else "vadusa_init"
            if self.ctx:
                self.L.vadusa_destroy(self.ctx)
                self.ctx = C.c_void_p()
            raise VadusaError(st, msg)
        self.batch = 0
        self.n_nodes = 0
        self._keep = {}

    def close(self):
        if getattr(self, "ctx", None):
            self.torch.cuda.synchronize(self.dev)
            self.L.vadusa_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, st: int):
        if st:
            raise VadusaError(st, self.L.vadusa_last_error(self.ctx).decode())

    def _enter(self):
        """Order the library's stream after the caller's current stream (inputs are ready)."""
        cur = self.torch.cuda.current_stream(self.dev)
        if cur != self.stream:
            self.stream.wait_stream(cur)

    def _leave(self):
        """Order the caller's current stream after the library's stream (outputs are ready)."""
        cur = self.torch.cuda.current_stream(self.dev)
        if cur != self.stream:
            cur.wait_stream(self.stream)

    @staticmethod
    def _p(t):
        return None if t is None else C.c_void_p(t.data_ptr())

    @staticmethod
    def _h(a: Optional[np.ndarray]):
        return None if a is None else a.ctypes.data_as(C.c_void_p)

    # ---- set-up ----
    def set_tree(self, parent: np.ndarray, rank: np.ndarray, per_sequence: bool = False):
        self._enter()
        parent = np.ascontiguousarray(parent, dtype=np.int32)
        rank = np.ascontiguousarray(rank, dtype=np.int32)
        n = parent.shape[-1]
        self._ck(self.L.vadusa_set_tree(self.ctx, n, self._h(parent), self._h(rank), int(per_sequence)))
        self.n_nodes = n
        self._leave()

    def begin(self, block_table, ctx_len: Optional[Sequence[int]] = None):
        """block_table: int32 [batch, max_blocks_per_seq] (numpy or device tensor)."""
        self._enter()
        torch = self.torch
        if not isinstance(block_table, torch.Tensor):
            bt = np.full((len(block_table), self.cfg.max_blocks_per_seq), -1, dtype=np.int32)
            src = np.asarray(block_table, dtype=np.int32)
            bt[:, :src.shape[1]] = src
            block_table = torch.from_numpy(bt).to(self.dev)
        self._keep["block_table"] = block_table
        self.batch = block_table.shape[0]
        cl = None if ctx_len is None else np.ascontiguousarray(ctx_len, dtype=np.int32)
        self._ck(self.L.vadusa_begin(self.ctx, self.batch, self._p(block_table), self._h(cl)))
        self._leave()

    def prefill(self, tokens: np.ndarray, lengths: Sequence[int]):
        self._enter()
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        lengths = np.ascontiguousarray(lengths, dtype=np.int32)
        self._ck(self.L.vadusa_prefill(self.ctx, self._h(tokens), self._h(lengths), tokens.shape[1]))
        self._leave()

    def load_state(self, hstar, logits_star):
        self._enter()
        self._ck(self.L.vadusa_load_state(self.ctx, self._p(hstar), self._p(logits_star)))
        self._leave()

    # ---- hot path ----
    def draft(self, sp: Sampling, tree_tokens=None, topk_out=None):
        self._enter()
        self._ck(self.L.vadusa_draft(self.ctx, C.byref(sp), self._p(tree_tokens), self._p(topk_out)))
        self._leave()

    def verify_step(self, override=None, logits_out=None, attn_tap=None, hidden_out=None):
        self._enter()
        self._ck(self.L.vadusa_verify_step(self.ctx, self._p(override), self._p(logits_out), self._p(attn_tap),
                                           self._p(hidden_out)))
        self._leave()

    def accept_and_commit(self, sp: Sampling, forced_best=None, accept_len=None, path_nodes=None, path_tokens=None,
                          kv_slots=None, edge_bits=None, next_root=None):
        self._enter()
        self._ck(self.L.vadusa_accept_and_commit(self.ctx, C.byref(sp), self._p(forced_best), self._p(accept_len),
                                                 self._p(path_nodes), self._p(path_tokens), self._p(kv_slots),
                                                 self._p(edge_bits), self._p(next_root)))
        self._leave()

    def generate(self, sp: Sampling, max_new_tokens: int, out_tokens, out_len, max_iters: int = 0) -> Stats:
        self._enter()
        st = Stats()
        self._ck(self.L.vadusa_generate(self.ctx, C.byref(sp), max_new_tokens, max_iters, self._p(out_tokens),
                                        self._p(out_len), C.byref(st)))
        self._leave()
        return st

    def generate_host(self, sp: Sampling, block_table, tokens: np.ndarray, lengths: np.ndarray,
                      max_new_tokens: int, out_tokens: np.ndarray, out_len: np.ndarray) -> Stats:
        """Host buffers in, host buffers out (block_table is a device tensor)."""
        self._enter()
        st = Stats()
        self._keep["block_table"] = block_table
        self.batch = block_table.shape[0]
        self._ck(self.L.vadusa_generate_host(self.ctx, C.byref(sp), self.batch, self._p(block_table), self._h(tokens),
                                             self._h(lengths), tokens.shape[1], max_new_tokens, self._h(out_tokens),
                                             self._h(out_len), C.byref(st)))
        self._leave()
        return st

    # ---- state ----
    def lengths(self) -> np.ndarray:
        out = np.zeros(self.batch, dtype=np.int32)
        self._ck(self.L.vadusa_get_lengths(self.ctx, self._h(out)))
        return out

    def check(self):
        self._ck(self.L.vadusa_check(self.ctx))

    def set_logit_bias(self, bias=None):
        """bias: fp32 device tensor [batch][>= vocab] added to the base head's logits when sampling, or None."""
        self._keep["logit_bias"] = bias
        self._ck(self.L.vadusa_set_logit_bias(self.ctx, self._p(bias), 0 if bias is None else bias.shape[1]))

    def accept_stats(self, reset: bool = False):
        """(tested, accepted) int64 [MAX_DEPTH][MAX_DRAFT_TOPK]: acceptance tests by (draft head, rank)."""
        t = np.zeros((MAX_DEPTH, MAX_DRAFT_TOPK), dtype=np.int64)
        a = np.zeros((MAX_DEPTH, MAX_DRAFT_TOPK), dtype=np.int64)
        self._ck(self.L.vadusa_accept_stats(self.ctx, self._h(t), self._h(a), int(reset)))
        return t, a

    def kernel_launches(self) -> int:
        return int(self.L.vadusa_kernel_launches(self.ctx))

    def set_fused_pass(self, enable):
        """False / True, or 6 / 8 to ask for that cluster size."""
        self._ck(self.L.vadusa_set_fused_pass(self.ctx, int(enable)))

    def set_attention_stream(self, enable):
        """Batches: True page-stream attention kernel, False (default) one thread block per (head, sequence)."""
        self._ck(self.L.vadusa_set_attention_stream(self.ctx, int(bool(enable))))

    def fused_pass_clusters(self) -> int:
        return int(self.L.vadusa_fused_pass_clusters(self.ctx))

    # ---- draft-head fitting ----
    def fit_begin(self, max_tokens: int, lam: float = 0.8, lr: float = 0.002, warmup: int = 40):
        n = self.L.vadusa_fit_state_bytes(C.byref(self.cfg), max_tokens)
        self._keep["fit_state"] = self.torch.zeros(n, dtype=self.torch.uint8, device=self.dev)
        self._enter()
        self._ck(self.L.vadusa_fit_begin(self.ctx, self._p(self._keep["fit_state"]), n, max_tokens, lam, lr, warmup))
        self._leave()

    def fit_step(self, hidden, targets, loss_out=None):
        self._enter()
        self._ck(self.L.vadusa_fit_step(self.ctx, self._p(hidden), self._p(targets), hidden.shape[0], self._p(loss_out)))
        self._leave()

    def fit_end(self):
        self._ck(self.L.vadusa_fit_end(self.ctx))
        self._keep.pop("fit_state", None)

    def set_prefill_tap(self, hidden_out=None):
        """hidden_out: device tensor [batch][stride][d_model] in the model dtype, or None."""
        self._keep["prefill_tap"] = hidden_out
        self._ck(self.L.vadusa_set_prefill_tap(self.ctx, self._p(hidden_out), 0 if hidden_out is None else hidden_out.shape[1]))

    def profile_begin(self):
        self._ck(self.L.vadusa_profile_begin(self.ctx))

    def profile_end(self) -> Dict[str, tuple]:
        """{kernel class: (launches, total_ms)} since profile_begin."""
        arr = (KernelTime * 32)()
        n = C.c_int32(0)
        self._ck(self.L.vadusa_profile_end(self.ctx, arr, 32, C.byref(n)))
        return {arr[i].name.decode(): (int(arr[i].launches), float(arr[i].total_ms)) for i in range(n.value)}

    # ---- helpers for tests and benchmarks: views of the caller-owned KV pool ----
    def kv_view(self):
        """The pool as a tensor [layers, blocks, 2, heads, 64, head_dim] of the model dtype."""
        c = self.cfg
        return self.kv_pool.view(self.tdtype).view(c.n_layers, c.kv_num_blocks, 2, c.n_heads, 64, c.d_model // c.n_heads)
