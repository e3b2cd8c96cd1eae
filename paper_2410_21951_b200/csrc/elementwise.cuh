// Tree build + embedding, LayerNorm (steps "tree build", "embed" and the LayerNorms of the verify pass).
#pragma once
#include "common.cuh"

namespace vadusa {

// One block per tree node row m = b * n_nodes + n.
// token = override ? override[m] : (n == 0 ? root[b] : topk[b][depth-1][rank]);
// position = ctx_len[b] + depth[n]; x[m] = E[token] + P[position] (fp32); kv_row[m] = cache slot of the node.
// Token ids >= vocab address the phoneme table.
template <typename T>
__global__ void tree_embed_kernel(TreeView tree, const int32_t* __restrict__ override_tokens,
                                  const int32_t* __restrict__ root, const int32_t* __restrict__ topk,
                                  int n_draft_heads, int draft_topk,
                                  const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ nvalid,
                                  const T* __restrict__ emb_audio, const T* __restrict__ emb_phon,
                                  const T* __restrict__ pos_table, int vocab, int n_phonemes, int max_pos, int d,
                                  int32_t* __restrict__ tokens_out, float* __restrict__ x,
                                  const int32_t* __restrict__ block_table, KvGeom geom, long long* __restrict__ kv_row,
                                  float2* __restrict__ stats /*[rows][d/128] or null*/, uint32_t* err) {
  const int m = blockIdx.x;
  const int b = m / tree.n_nodes, n = m % tree.n_nodes;
  const int to = tree.off(b);
  const int depth = tree.depth[to + n];
  int tok;
  if (override_tokens) tok = override_tokens[m];
  else if (n == 0) tok = root[b];
  else tok = topk[(b * n_draft_heads + (depth - 1)) * draft_topk + tree.rank[to + n]];
  const bool live = n < nvalid[b];
  if (!live) tok = 0;
  int pos = ctx_len[b] + depth;
  if (pos >= max_pos) { if (live && threadIdx.x == 0) atomicOr(err, kErrCapacity); pos = max_pos - 1; }
  const T* e;
  if (tok >= 0 && tok < vocab) e = emb_audio + (long long)tok * d;
  else if (tok >= vocab && tok < vocab + n_phonemes) e = emb_phon + (long long)(tok - vocab) * d;
  else { if (live && threadIdx.x == 0) atomicOr(err, kErrCapacity); e = emb_audio; }
  if (threadIdx.x == 0) {
    tokens_out[m] = tok;
    // where this node's K/V rows go: slot ctx_len + n behind the context (the q/k/v product's
    // epilogue reads this instead of walking the block table per element)
    long long row = -1;
    if (live && kv_row) {
      const int slot = ctx_len[b] + n;
      const long long blk = kv_block_of(block_table, geom, b, slot, err);
      if (blk >= 0) row = geom.elem(blk, 0, 0, slot % kKvBlock);
    }
    if (kv_row) kv_row[m] = row;
  }
  const T* p = pos_table + (long long)pos * d;
  if (stats) {
    // d is a multiple of 128: warp w takes the groups of 128 features w, w + 4, ... (lane l: features 4l .. 4l+3 of
    // the group) and leaves each group's mean and sum of squared deviations for the LayerNorm folded into the
    // first product
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nt = d >> 7;
    for (int gi = warp; gi < nt; gi += (int)(blockDim.x >> 5)) {
      const int c0 = 128 * gi + 4 * lane;
      float4 v;
      v.x = to_f<T>(e[c0]) + to_f<T>(p[c0]);         v.y = to_f<T>(e[c0 + 1]) + to_f<T>(p[c0 + 1]);
      v.z = to_f<T>(e[c0 + 2]) + to_f<T>(p[c0 + 2]); v.w = to_f<T>(e[c0 + 3]) + to_f<T>(p[c0 + 3]);
      *reinterpret_cast<float4*>(x + (long long)m * d + c0) = v;
      const float mu = warp_sum((v.x + v.y) + (v.z + v.w)) * (1.0f / 128.0f);
      const float d0 = v.x - mu, d1 = v.y - mu, d2 = v.z - mu, d3 = v.w - mu;
      const float q = warp_sum((d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3));
      if (lane == 0) stats[(long long)m * nt + gi] = make_float2(mu, q);
    }
    return;
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) x[(long long)m * d + i] = to_f<T>(e[i]) + to_f<T>(p[i]);
}

// order[r] = the sequence with the r-th longest context (ties: lower index first); inactive
// sequences last.  The attention grid visits sequences in this order, so the longest chains
// start first and a ragged batch balances over the SMs.  One block.
__global__ void seq_order_kernel(const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ nvalid, int batch,
                                 int32_t* __restrict__ order) {
  for (int b = threadIdx.x; b < batch; b += blockDim.x) {
    const int lb = nvalid[b] > 0 ? ctx_len[b] : -1;
    int rank = 0;
    for (int o = 0; o < batch; ++o) {
      const int lo = nvalid[o] > 0 ? ctx_len[o] : -1;
      rank += (lo > lb || (lo == lb && o < b)) ? 1 : 0;
    }
    order[rank] = b;
  }
}

// One block per row: y = (x - mean) / sqrt(var + eps) * g + b, rounded to T.  The row is read
// once into registers (up to 8 values per thread, d <= 8 * blockDim.x).
template <typename T>
__global__ void __launch_bounds__(256) layernorm_kernel(const float* __restrict__ x, const float* __restrict__ g,
                                                        const float* __restrict__ bta, T* __restrict__ y, int rows, int d,
                                                        float eps) {
  __shared__ float red[8];
  // launched as a programmatic dependent: let the next kernel start its prologue, then wait
  // for the producer of x
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.x;
  const float* xr = x + (long long)row * d;
  float v[8];
  int cnt = 0;
  float s = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { v[cnt] = xr[i]; s += v[cnt]; ++cnt; }
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];
  const float mean = tot / (float)d;
  __syncthreads();
  float q = 0.f;
  for (int c = 0; c < cnt; ++c) { const float t = v[c] - mean; q += t * t; }
  q = warp_sum(q);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = q;
  __syncthreads();
  float var = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) var += red[w];
  const float rstd = 1.0f / sqrtf(var / (float)d + eps);
  T* yr = y + (long long)row * d;
  cnt = 0;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { yr[i] = from_f<T>((v[cnt] - mean) * rstd * g[i] + bta[i]); ++cnt; }
}

// The same LayerNorm with one warp per row, for rows whose length is a multiple of 128 (up to 2048): lane l
// holds columns 128 j + 4 l .. + 3 of the row in registers (all loads issued at once), the two sums go through
// warp shuffles, and the result is written four values at a time.  8 rows per block of 256 threads.
template <typename T>
__global__ void __launch_bounds__(256) layernorm_rows_kernel(const float* __restrict__ x, const float* __restrict__ g,
                                                             const float* __restrict__ bta, T* __restrict__ y, int rows,
                                                             int d, float eps) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int nj = d >> 7;
  const float4* xr = reinterpret_cast<const float4*>(x + (long long)row * d);
  float4 v[16];
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if (j < nj) v[j] = xr[32 * j + lane];
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if (j < nj) s += (v[j].x + v[j].y) + (v[j].z + v[j].w);
  s = warp_sum(s);
  // the rows are in registers: the next kernel may start (all blocks of this grid fit on the GPU at once, so
  // an earlier signal would let it take the SMs while the kernel before this one is still running)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const float mean = s / (float)d;
  float q = 0.f;
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if (j < nj) {
      const float a = v[j].x - mean, b = v[j].y - mean, c = v[j].z - mean, e = v[j].w - mean;
      q += (a * a + b * b) + (c * c + e * e);
    }
  q = warp_sum(q);
  const float rstd = 1.0f / sqrtf(q / (float)d + eps);
  T* yr = y + (long long)row * d;
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if (j < nj) {
      const int c0 = 128 * j + 4 * lane;
      const float4 gg = *reinterpret_cast<const float4*>(g + c0), bb = *reinterpret_cast<const float4*>(bta + c0);
      store4<T>(yr + c0, (v[j].x - mean) * rstd * gg.x + bb.x, (v[j].y - mean) * rstd * gg.y + bb.y,
                (v[j].z - mean) * rstd * gg.z + bb.z, (v[j].w - mean) * rstd * gg.w + bb.w);
    }
}

}  // namespace vadusa
