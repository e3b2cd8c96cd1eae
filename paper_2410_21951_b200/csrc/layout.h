// Host-side layout arithmetic: weight blob, workspace, KV pool.  No CUDA calls.
#pragma once
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <vector>

#include "../../include/vadusa.h"

namespace vadusa {

constexpr int64_t kLnStatsBytes = 64 * 8 * 8;     // [token <= 64][feature group <= 8] (mean, sum of squared deviations)
constexpr int64_t kGemmPartBytes = 32ll << 20;   // split-K exchange area (a launch needs tiles * ksplit * TN * 128 * 4 bytes)
constexpr int kGenHostCap = 4096;     // most tokens per sequence vadusa_generate_host can return

inline int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

inline const char* check_config(const vadusa_config* c) {
  if (!c) return "config is NULL";
  if (c->struct_size != sizeof(vadusa_config)) return "config.struct_size does not match this library";
  if (c->abi_version != VADUSA_ABI_VERSION) return "config.abi_version does not match this library";
  if (c->dtype != 0 && c->dtype != 1) return "dtype must be 0 (fp32) or 1 (bf16)";
  if (c->n_layers < 1 || c->n_layers > 64) return "n_layers out of range";
  if (c->d_model < 64 || c->d_model % 64 || c->d_model > 2048) return "d_model must be a multiple of 64 in 64..2048";
  if (c->n_heads < 1 || c->d_model % c->n_heads) return "n_heads must divide d_model";
  {
    int dh = c->d_model / c->n_heads;
    if (dh != 32 && dh != 64) return "head_dim must be 32 or 64";
  }
  if (c->d_ffn < 16 || c->d_ffn % 16) return "d_ffn must be a positive multiple of 16";
  if (c->vocab < 2 || c->vocab > 24576) return "vocab must be in 2..24576 (two rows of it live in shared memory)";
  if (c->n_phonemes < 0) return "n_phonemes must be >= 0";
  if (c->max_pos < 1) return "max_pos must be positive";
  if (c->n_draft_heads < 1 || c->n_draft_heads > VADUSA_MAX_DEPTH) return "n_draft_heads out of range";
  if (c->draft_topk < 1 || c->draft_topk > VADUSA_MAX_DRAFT_TOPK || c->draft_topk >= c->vocab)
    return "draft_topk out of range";
  if (c->max_batch < 1 || c->max_batch > 4096) return "max_batch out of range";
  if (c->max_tree_nodes < 1 || c->max_tree_nodes > VADUSA_MAX_TREE_NODES) return "max_tree_nodes out of range";
  if (c->kv_block != 64) return "kv_block must be 64";
  if (c->max_blocks_per_seq < 1) return "max_blocks_per_seq must be positive";
  if (c->prefill_rows < 0 || c->prefill_rows > 4096) return "prefill_rows out of range";
  if (c->reserved0 != 0) return "reserved0 must be 0";
  if (c->kv_num_blocks < 1) return "kv_num_blocks must be positive";
  if (!(c->ln_eps > 0.f)) return "ln_eps must be positive";
  return nullptr;
}

inline int esize(const vadusa_config* c) { return c->dtype == 1 ? 2 : 4; }
// Rows (sequences, or prefix chunks during prefill) of max_tree_nodes tokens that one pass through the model holds.
inline int pass_rows(const vadusa_config* c) { return c->prefill_rows > c->max_batch ? c->prefill_rows : c->max_batch; }
inline int vpad(const vadusa_config* c) { return (int)align_up(c->vocab, 128); }

struct TensorDesc {
  std::string name;
  int64_t offset, nbytes;
  int rows, cols, rows_padded, is_matrix;
};

// Order: embeddings, layers, final norm, base head, then the draft heads grouped by kind
// (all W, all b, all U) so that a batched product over heads sees a constant stride.
inline std::vector<TensorDesc> weight_layout(const vadusa_config* c, int64_t* total) {
  std::vector<TensorDesc> v;
  int64_t off = 0;
  const int es = esize(c), d = c->d_model, f = c->d_ffn;
  auto mat = [&](const std::string& n, int rows, int cols, int rows_padded) {
    int64_t nb = (int64_t)rows_padded * cols * es;
    v.push_back({n, off, nb, rows, cols, rows_padded, 1});
    off = align_up(off + nb, 256);
  };
  auto vec = [&](const std::string& n, int rows) {
    int64_t nb = (int64_t)rows * 4;
    v.push_back({n, off, nb, rows, 1, rows, 0});
    off = align_up(off + nb, 256);
  };
  mat("emb_audio", c->vocab, d, c->vocab);
  mat("emb_phon", c->n_phonemes > 0 ? c->n_phonemes : 1, d, c->n_phonemes > 0 ? c->n_phonemes : 1);
  mat("pos", c->max_pos, d, c->max_pos);
  for (int l = 0; l < c->n_layers; ++l) {
    std::string p = "l" + std::to_string(l) + ".";
    vec(p + "ln1_g", d); vec(p + "ln1_b", d);
    mat(p + "wqkv", 3 * d, d, 3 * d); vec(p + "bqkv", 3 * d);
    mat(p + "wo", d, d, d); vec(p + "bo", d);
    vec(p + "ln2_g", d); vec(p + "ln2_b", d);
    mat(p + "w1", f, d, f); vec(p + "b1", f);
    mat(p + "w2", d, f, d); vec(p + "b2", d);
  }
  vec("lnf_g", d); vec("lnf_b", d);
  mat("lm", c->vocab, d, vpad(c));
  for (int i = 0; i < c->n_draft_heads; ++i) mat("draft" + std::to_string(i) + ".w", d, d, d);
  for (int i = 0; i < c->n_draft_heads; ++i) vec("draft" + std::to_string(i) + ".b", d);
  for (int i = 0; i < c->n_draft_heads; ++i) mat("draft" + std::to_string(i) + ".u", c->vocab, d, vpad(c));
  if (total) *total = off;
  return v;
}

struct WorkspaceLayout {
  int64_t scalars;                       // uint32 err, int32 done_count, padding
  int64_t ctx_len, nvalid, gen_count, commit_base, commit_len, best, root, saved_nvalid;   // int32 [B]
  int64_t commit_path;                   // int32 [B][16]
  int64_t seq_order;                     // int32 [R]: rows by descending context length
  int64_t tree_parent, tree_depth, tree_rank, tree_anc;       // [B*128] (anc: two uint64 per node)
  int64_t chain_parent, chain_depth, chain_rank, chain_anc;   // [128]
  int64_t tokens, stage_tokens;          // int32 [M]
  int64_t kv_row;                        // int64 [M]: element offset of the row's K slot (head 0) in a layer's pool, -1: none
  int64_t topk;                          // int32 [B][heads][k]
  int64_t x;                             // fp32 [M][d]
  int64_t a, q, o, hfinal;               // T [M][d]
  int64_t mid;                           // T [M][f]
  int64_t logits;                        // fp32 [M][vpad]
  int64_t hstar, logits_star;            // T [B][d], fp32 [B][vpad]
  int64_t z, dlogits;                    // T [heads][B][d], fp32 [heads][B][vpad]
  int64_t att_xch;                       // fp32 split-KV exchange of the attention kernels: 592 slots of 64*64+128 floats
  int64_t att_cnt;                       // uint32 [592]: parts of an item that have arrived (page-stream attention); zero between launches
  int64_t gemm_part;                     // fp32 split-K exchange of the tensor-core products (kGemmPartBytes)
  int64_t ln_stats;                      // per-group LayerNorm statistics for the fused products (kLnStatsBytes)
  int64_t acc_stats;                     // uint64 [2][VADUSA_MAX_DEPTH][VADUSA_MAX_DRAFT_TOPK]: edges tested, edges accepted
  int64_t gen_out, gen_len;              // int32 [B][kGenHostCap], int32 [B] (vadusa_generate_host staging)
  // prefill: one row per prefix chunk of a pass (R = pass_rows)
  int64_t pf_ctx_len, pf_nvalid, pf_seq, pf_last;   // int32 [R]: tokens before the chunk, its length, its sequence, sequence if last chunk else -1
  int64_t pf_block_table;                // int32 [R][max_blocks_per_seq]: the block-table row of the chunk's sequence
  int64_t pf_pairs;                      // int2 [R]: rows that share an attention CTA during prefill (y < 0: a single chunk)
  // single-sequence pass in one persistent kernel: residual stream after the attention block, LayerNorm statistics
  // per (token, group of 64 features) of both residual buffers, counters of the exchanges between clusters
  int64_t f_xb, f_stats_a, f_stats_b, f_sync;    // fp32 [64][d], float2 [64][d/64] x 2, uint32 [64]
  int64_t total;
};

inline WorkspaceLayout workspace_layout(const vadusa_config* c) {
  WorkspaceLayout w;
  int64_t off = 0;
  const int64_t B = c->max_batch, R = pass_rows(c), N = c->max_tree_nodes, M = R * N, d = c->d_model, f = c->d_ffn;
  const int64_t es = esize(c), vp = vpad(c), hd = c->n_draft_heads;
  auto take = [&](int64_t bytes) { int64_t o = off; off = align_up(off + bytes, 256); return o; };
  w.scalars = take(256);
  w.ctx_len = take(B * 4); w.nvalid = take(B * 4); w.gen_count = take(B * 4);
  w.commit_base = take(B * 4); w.commit_len = take(B * 4); w.best = take(B * 4); w.root = take(B * 4);
  w.saved_nvalid = take(B * 4);
  w.commit_path = take(B * 16 * 4);
  w.seq_order = take(R * 4);
  const int64_t T = VADUSA_MAX_TREE_NODES;
  w.tree_parent = take(B * T * 4); w.tree_depth = take(B * T * 4); w.tree_rank = take(B * T * 4);
  w.tree_anc = take(B * T * 16);
  w.chain_parent = take(T * 4); w.chain_depth = take(T * 4); w.chain_rank = take(T * 4);
  w.chain_anc = take(T * 16);
  w.tokens = take(M * 4); w.stage_tokens = take(M * 4);
  w.kv_row = take(M * 8);
  w.topk = take(B * hd * c->draft_topk * 4);
  w.x = take(M * d * 4);
  w.a = take(M * d * es); w.q = take(M * d * es); w.o = take(M * d * es); w.hfinal = take(M * d * es);
  w.mid = take(M * f * es);
  w.logits = take(M * vp * 4);
  w.hstar = take(B * d * es); w.logits_star = take(B * vp * 4);
  w.z = take(hd * B * d * es); w.dlogits = take(hd * B * vp * 4);
  w.att_xch = take(592ll * (64 * 64 + 128) * 4);
  w.att_cnt = take(592 * 4);
  w.gemm_part = take(kGemmPartBytes);
  w.ln_stats = take(kLnStatsBytes);
  w.acc_stats = take(2ll * VADUSA_MAX_DEPTH * VADUSA_MAX_DRAFT_TOPK * 8);
  w.gen_out = take(B * kGenHostCap * 4); w.gen_len = take(B * 4);
  w.pf_ctx_len = take(R * 4); w.pf_nvalid = take(R * 4); w.pf_seq = take(R * 4); w.pf_last = take(R * 4);
  w.pf_block_table = take(R * (int64_t)c->max_blocks_per_seq * 4);
  w.pf_pairs = take(R * 8);
  w.f_xb = take(64 * d * 4);
  w.f_stats_a = take(64 * (d / 64 + 1) * 8); w.f_stats_b = take(64 * (d / 64 + 1) * 8);
  w.f_sync = take(256);
  w.total = off;
  return w;
}

inline int64_t kv_pool_bytes(const vadusa_config* c) {
  return (int64_t)c->n_layers * c->kv_num_blocks * 2 * c->d_model * 64 * esize(c);
}

}  // namespace vadusa
