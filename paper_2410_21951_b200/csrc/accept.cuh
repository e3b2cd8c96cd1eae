// Tolerance verification (Algorithm 1), choice of the longest / leftmost accepted
// path (Sec. II-C) and the commit of its K/V rows into the cache.
#pragma once
#include "select.cuh"

namespace vadusa {

struct AcceptOut {            // optional user-visible outputs (any may be null)
  int32_t* accept_len;        // [batch]
  int32_t* path_nodes;        // [batch][kMaxPath]
  int32_t* path_tokens;       // [batch][kMaxPath]
  long long* kv_slots;        // [batch][kMaxPath]
  unsigned long long* edge_bits;  // [batch][edge_words]
  long long edge_words;       // 1 (trees of up to 64 nodes) or 2 (a full word: the struct's bytes key the graph cache)
  int32_t* next_root;         // [batch]
};

struct SeqState {             // device state of the batch (all [batch] unless noted)
  int32_t* ctx_len;
  int32_t* nvalid;            // tree nodes scored for the sequence this iteration (0: inactive)
  int32_t* gen_count;         // tokens generated so far
  int32_t* commit_base;       // context length before the commit
  int32_t* commit_len;        // accepted length
  int32_t* commit_path;       // [batch][kMaxPath] node ids of the winning path
  int32_t* best;              // winning node
  int32_t* out_tokens;        // [batch][out_cap] generated tokens (may be null)
  int32_t* done_count;        // scalar: sequences that reached the target
  int out_cap;
  int target;                 // stop a sequence after this many tokens (0: never)
  unsigned long long* stats;  // [2][kStatDepth][kStatTopk]: acceptance tests applied / passed, by (draft head, rank)
};


// One block per sequence.  A sequence whose path commits EOS (when EOS is not masked) or reaches the token
// target becomes inactive (nvalid = 0).  Edges are tested depth by depth, only below accepted nodes:
// for an accepted parent p the keys of its logits row are formed once in shared memory
// (they predict absolute position ctx_len + depth(p) + 1), then each child token c is
// accepted iff fewer than tau tokens precede it in key order (and it lies in the nucleus).
// dynamic shared memory: 2 * ld floats.
__global__ void __launch_bounds__(256) accept_kernel(
    const float* __restrict__ logits, int ld, int vocab, const int32_t* __restrict__ tokens, TreeView tree,
    const int32_t* __restrict__ block_table, KvGeom geom, SamplingDev sp,
    const int32_t* __restrict__ forced_best, SeqState st, AcceptOut out, uint32_t* err) {
  extern __shared__ float keys[];          // [ld] keys, then [ld] probabilities (nucleus only)
  float* probs = keys + ld;
  __shared__ int s_parent[kMaxNodes], s_depth[kMaxNodes], s_tok[kMaxNodes];
  __shared__ int s_child[kMaxNodes], s_ok[kMaxNodes], s_nchild;
  __shared__ unsigned long long s_edges[2], s_acc[2];    // bits 0..63, 64..127
  __shared__ int s_path[kMaxPath], s_best, s_len, s_eos;
  __shared__ int s_first[kMaxPath + 2];    // nodes are ordered by depth: first node of every depth, then nv
  __shared__ Best bscratch[32];
  __shared__ float fscratch[32];
  __shared__ int s_scan[256];

  const int b = blockIdx.x, N = tree.n_nodes, nv = st.nvalid[b];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (nv == 0) {
    if (tid == 0) {
      st.commit_len[b] = 0;
      if (out.accept_len) out.accept_len[b] = 0;
      if (out.edge_bits) for (int w = 0; w < (int)out.edge_words; ++w) out.edge_bits[b * out.edge_words + w] = 0ull;
      if (out.next_root) out.next_root[b] = -1;
    }
    if (tid < kMaxPath) {
      if (out.path_nodes) out.path_nodes[b * kMaxPath + tid] = -1;
      if (out.path_tokens) out.path_tokens[b * kMaxPath + tid] = -1;
      if (out.kv_slots) out.kv_slots[b * kMaxPath + tid] = -1;
    }
    return;
  }
  const int S = st.ctx_len[b];
  const int to = tree.off(b);
  if (tid < kMaxNodes) {
    const bool in = tid < nv;
    s_parent[tid] = in ? tree.parent[to + tid] : -1;
    s_depth[tid] = in ? tree.depth[to + tid] : -1;
    s_tok[tid] = in ? tokens[(long long)b * N + tid] : -1;
  }
  if (tid == 0) { s_edges[0] = 1ull; s_acc[0] = 1ull; s_edges[1] = 0ull; s_acc[1] = 0ull; }
  if (tid < kMaxPath + 2) s_first[tid] = nv;
  __syncthreads();
  if (tid < nv && (tid == 0 || s_depth[tid] != s_depth[tid - 1])) s_first[min(s_depth[tid], kMaxPath)] = tid;
  __syncthreads();
  const int maxdepth = min(s_depth[nv - 1], kMaxPath - 1);
  const bool nuc = nucleus_on(sp);
  const int fb = forced_best ? forced_best[b] : -1;

  for (int d = 0; d < maxdepth && fb < 0; ++d) {
    __syncthreads();                               // the accepted set of depth d is final
    const unsigned long long a0 = s_acc[0], a1 = s_acc[1];
    const int p_end = s_first[d + 1];
    bool any = false;
    for (int p = s_first[d]; p < p_end; ++p) {
      if (!bit_at(a0, a1, p)) continue;            // uniform
      any = true;
      __syncthreads();
      if (tid == 0) s_nchild = 0;
      __syncthreads();
      if (tid < nv && s_parent[tid] == p) s_child[atomicAdd(&s_nchild, 1)] = tid;
      __syncthreads();
      const int nchild = s_nchild;
      if (nchild == 0) continue;
      const BaseRow row = base_row(logits + ((long long)b * N + p) * ld, sp, b);
      const uint64_t rs = noise_row_state(sp.seed, b, S + d + 1);
      const bool noise = sp.accept_rule == 0;
      for (int j = tid; j < vocab; j += blockDim.x) keys[j] = key_of(row[j], j, rs, sp, noise);
      if (nuc) {
        // Tokens outside the top-p nucleus cannot be drawn: give them the key -inf.  In the order "larger logit,
        // then lower id" the nucleus is the prefix of tokens whose mass ahead of them is below top_p.  The mass
        // strictly above a logit value falls as the value grows, so the smallest value v* whose mass above is
        // still below top_p is found by bisection on the ordered bit pattern of the value (32 block-wide sums
        // instead of one pass per token); tokens above v* are inside, tokens below it outside, and the tokens
        // AT v* (equal logits, equal probability p*) are inside while (mass above v*) + (ties with a lower
        // id) * p* stays below top_p.  probs[] holds exp((l - max) / T).
        const RowStats rst = row_stats(row, vocab, sp, fscratch);
        for (int j = tid; j < vocab; j += blockDim.x)
          probs[j] = expf((masked_logit(row[j], j, sp) - rst.maxl) * sp.inv_temperature);
        __syncthreads();
        const float limit = sp.top_p * rst.z;
        auto mass_above = [&](uint32_t k) -> float {              // sum of p over tokens whose value orders above k
          float m = 0.f;
          for (int j = tid; j < vocab; j += blockDim.x)
            if (ordered_bits(masked_logit(row[j], j, sp)) > k) m += probs[j];
          return block_sum(m, fscratch);
        };
        uint32_t lo = 0u, hi = 0xffffffffu;                       // mass_above(hi) = 0 < limit: v* in (lo, hi]
        if (mass_above(0u) < limit) hi = 0u;                      // (everything is inside)
        while (hi - lo > 1u) {
          const uint32_t mid = lo + ((hi - lo) >> 1);
          if (mass_above(mid) < limit) hi = mid; else lo = mid;
        }
        const float above = mass_above(hi);
        // ties at v*: exclusive count of earlier ids with the same value, by contiguous chunks of ids
        const int chunk = (vocab + (int)blockDim.x - 1) / (int)blockDim.x, j0 = tid * chunk, j1 = min(vocab, j0 + chunk);
        int mine = 0;
        for (int j = j0; j < j1; ++j) mine += ordered_bits(masked_logit(row[j], j, sp)) == hi ? 1 : 0;
        __syncthreads();
        s_scan[tid] = mine;
        __syncthreads();
        int before = 0;
        for (int t = 0; t < tid; ++t) before += s_scan[t];
        for (int j = j0; j < j1; ++j) {
          const uint32_t kj = ordered_bits(masked_logit(row[j], j, sp));
          bool inside = kj > hi;
          if (kj == hi) { inside = above + (float)before * probs[j] < limit; ++before; }
          if (!inside) keys[j] = -INFINITY;
        }
      }
      __syncthreads();
      for (int i = warp; i < nchild; i += (blockDim.x >> 5)) {
        const int c = s_tok[s_child[i]];
        int cnt = sp.tau;                                            // not a speech token: never accepted
        bool finite = false;
        if (c >= 0 && c < vocab) {
          const float kc = keys[c];
          finite = kc > -INFINITY;
          cnt = 0;
          for (int j = lane; j < vocab; j += 32) cnt += precedes(keys[j], j, kc, c) ? 1 : 0;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        }
        if (lane == 0) s_ok[i] = (cnt < sp.tau && finite) ? 1 : 0;
      }
      __syncthreads();
      if (tid == 0) {
        for (int i = 0; i < nchild; ++i)
          if (s_ok[i]) { const int c = s_child[i]; s_edges[c >> 6] |= 1ull << (c & 63); s_acc[c >> 6] |= 1ull << (c & 63); }
      }
      if (tid < nchild && st.stats && d < kStatDepth) {
        const int r = tree.rank[to + s_child[tid]];
        if (r >= 0 && r < kStatTopk) {
          atomicAdd(st.stats + d * kStatTopk + r, 1ull);
          if (s_ok[tid]) atomicAdd(st.stats + (kStatDepth + d) * kStatTopk + r, 1ull);
        }
      }
      __syncthreads();
    }
    if (!any) break;                               // nothing accepted at this depth: nothing below it either
  }
  __syncthreads();
  if (tid == 0) {
    int best = 0;
    if (fb >= 0 && fb < nv) best = fb;
    else {
      // deepest accepted node, the first (leftmost) of that depth
      const unsigned long long a0 = s_acc[0], a1 = s_acc[1];
      for (int d = maxdepth; d >= 1 && best == 0; --d)
        for (int n = s_first[d]; n < s_first[d + 1]; ++n)
          if (bit_at(a0, a1, n)) { best = n; break; }
    }
    int len = min(s_depth[best] + 1, kMaxPath);
    int n = best;
    for (int j = len - 1; j >= 0; --j) { s_path[j] = n; n = s_parent[n]; }
    // EOS not masked: the sequence ends with the first EOS on the path; what follows it is dropped
    s_eos = 0;
    if (!sp.eos_masked)
      for (int j = 0; j < len; ++j)
        if (s_tok[s_path[j]] == sp.eos_id) { len = j + 1; best = s_path[j]; s_eos = 1; break; }
    s_best = best; s_len = len;
  }
  __syncthreads();
  const int best = s_best, len = s_len;
  const int nroot = sample_row(base_row(logits + ((long long)b * N + best) * ld, sp, b), vocab, b, S + len, sp, bscratch, fscratch);

  if (tid < kMaxPath) {
    const bool in = tid < len;
    const int node = in ? s_path[tid] : -1;
    st.commit_path[b * kMaxPath + tid] = node;
    long long slot = -1;
    if (in) {
      const long long blk = kv_block_of(block_table, geom, b, S + tid, err);
      slot = blk < 0 ? -1 : blk * kKvBlock + (S + tid) % kKvBlock;
    }
    if (out.path_nodes) out.path_nodes[b * kMaxPath + tid] = node;
    if (out.path_tokens) out.path_tokens[b * kMaxPath + tid] = in ? s_tok[node] : -1;
    if (out.kv_slots) out.kv_slots[b * kMaxPath + tid] = slot;
    if (in && st.out_tokens) {
      const int g = st.gen_count[b] + tid;
      if (g < st.out_cap) st.out_tokens[(long long)b * st.out_cap + g] = s_tok[node];
    }
  }
  __syncthreads();
  if (tid == 0) {
    st.commit_base[b] = S;
    st.commit_len[b] = len;
    st.best[b] = best;
    st.ctx_len[b] = S + len;
    const int g = st.gen_count[b] + len;
    st.gen_count[b] = g;
    if (s_eos || (st.target > 0 && g >= st.target)) { st.nvalid[b] = 0; atomicAdd(st.done_count, 1); }
    if (out.accept_len) out.accept_len[b] = len;
    if (out.edge_bits) for (int w = 0; w < (int)out.edge_words; ++w) out.edge_bits[b * out.edge_words + w] = s_edges[w];
    if (out.next_root) out.next_root[b] = nroot;
  }
}

// grid = (n_layers + 1, batch).  x < n_layers: move the K/V rows of the winning path of
// layer x from slot base + path[j] to slot base + j, 16 bytes per thread and step; a
// thread always handles the same 16-byte column of every row, and rows are taken in
// ascending j, so a destination is never read again after it was overwritten.
// x == n_layers: carry the winner's hidden state and logits.
template <typename T>
__global__ void __launch_bounds__(256) commit_kernel(
    T* __restrict__ pool, KvGeom geom, const int32_t* __restrict__ block_table, SeqState st,
    int n_layers, int n_nodes, const T* __restrict__ hfinal, int d_model, const float* __restrict__ logits, int ld,
    T* __restrict__ hstar, float* __restrict__ logits_star, uint32_t* err) {
  const int b = blockIdx.y, len = st.commit_len[b];
  if (len == 0) return;
  if ((int)blockIdx.x == n_layers) {
    const long long m = (long long)b * n_nodes + st.best[b];
    for (int i = threadIdx.x; i < d_model; i += blockDim.x) hstar[(long long)b * d_model + i] = hfinal[m * d_model + i];
    for (int i = threadIdx.x; i < ld; i += blockDim.x) logits_star[(long long)b * ld + i] = logits[m * ld + i];
    return;
  }
  __shared__ long long s_src[kMaxPath], s_dst[kMaxPath];
  const int base = st.commit_base[b];
  if (threadIdx.x < kMaxPath) {
    const int j = threadIdx.x;
    long long src = -1, dst = -1;
    if (j < len) {
      const int node = st.commit_path[b * kMaxPath + j];
      if (node != j) {
        const long long bs = kv_block_of(block_table, geom, b, base + node, err);
        const long long bd = kv_block_of(block_table, geom, b, base + j, err);
        if (bs >= 0 && bd >= 0) {
          src = geom.elem(bs, 0, 0, (base + node) % kKvBlock);
          dst = geom.elem(bd, 0, 0, (base + j) % kKvBlock);
        }
      }
    }
    s_src[j] = src; s_dst[j] = dst;
  }
  __syncthreads();
  T* lp = pool + (long long)blockIdx.x * geom.layer_stride;
  const int cpr = geom.head_dim * (int)sizeof(T) / 16;            // 16-byte chunks per row
  const int chunks = 2 * geom.n_heads * cpr;
  const long long row_stride = (long long)kKvBlock * geom.head_dim;   // elements between (kv, head) tiles
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    const int tile = c / cpr, cc = c % cpr;
    for (int j = 1; j < len; ++j) {
      if (s_src[j] < 0) continue;
      const uint4* s = reinterpret_cast<const uint4*>(lp + s_src[j] + tile * row_stride) + cc;
      uint4* dd = reinterpret_cast<uint4*>(lp + s_dst[j] + tile * row_stride) + cc;
      *dd = *s;
    }
  }
}

// Prefill bookkeeping.  gather: row r of the pass gets the block-table row of its sequence.
__global__ void prefill_gather_kernel(const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_of,
                                      int max_blocks, int32_t* __restrict__ out) {
  const int r = blockIdx.x, b = seq_of[r];
  for (int i = threadIdx.x; i < max_blocks; i += blockDim.x) out[(long long)r * max_blocks + i] = block_table[(long long)b * max_blocks + i];
}

// finish: the row holding the last chunk of sequence b carries that sequence's state forward: the
// hidden state and base-head logits of its last token, and the new context length.  grid = rows.
template <typename T>
__global__ void prefill_finish_kernel(const int32_t* __restrict__ row_ctx, const int32_t* __restrict__ row_nvalid,
                                      const int32_t* __restrict__ row_last, int n_nodes, const T* __restrict__ hfinal,
                                      int d_model, const float* __restrict__ logits, int ld, T* __restrict__ hstar,
                                      float* __restrict__ logits_star, int32_t* __restrict__ ctx_len) {
  const int r = blockIdx.x, b = row_last[r], nv = row_nvalid[r];
  if (b < 0 || nv == 0) return;
  const long long m = (long long)r * n_nodes + nv - 1;
  for (int i = threadIdx.x; i < d_model; i += blockDim.x) hstar[(long long)b * d_model + i] = hfinal[m * d_model + i];
  for (int i = threadIdx.x; i < ld; i += blockDim.x) logits_star[(long long)b * ld + i] = logits[m * ld + i];
  if (threadIdx.x == 0) ctx_len[b] = row_ctx[r] + nv;
}

}  // namespace vadusa
