// Tree build + embedding, LayerNorm (steps "tree build", "embed" and the LayerNorms of the verify pass).
#pragma once
#include "common.cuh"

namespace vadusa {

// One block per tree node row m = b * n_nodes + n.
// token = override ? override[m] : (n == 0 ? root[b] : topk[b][depth-1][rank]);
// position = ctx_len[b] + depth[n]; x[m] = E[token] + P[position] (fp32).
// Token ids >= vocab address the phoneme table.
template <typename T>
__global__ void tree_embed_kernel(TreeView tree, const int32_t* __restrict__ override_tokens,
                                  const int32_t* __restrict__ root, const int32_t* __restrict__ topk,
                                  int n_draft_heads, int draft_topk,
                                  const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ nvalid,
                                  const T* __restrict__ emb_audio, const T* __restrict__ emb_phon,
                                  const T* __restrict__ pos_table, int vocab, int n_phonemes, int max_pos, int d,
                                  int32_t* __restrict__ tokens_out, float* __restrict__ x, uint32_t* err) {
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
  if (threadIdx.x == 0) tokens_out[m] = tok;
  const T* p = pos_table + (long long)pos * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) x[(long long)m * d + i] = to_f<T>(e[i]) + to_f<T>(p[i]);
}

// One warp per row: y = (x - mean) / sqrt(var + eps) * g + b, rounded to T.
template <typename T>
__global__ void layernorm_kernel(const float* __restrict__ x, const float* __restrict__ g,
                                 const float* __restrict__ bta, T* __restrict__ y, int rows, int d, float eps) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float* xr = x + (long long)row * d;
  float s = 0.f;
  for (int i = lane; i < d; i += 32) s += xr[i];
  const float mean = warp_sum(s) / (float)d;
  float v = 0.f;
  for (int i = lane; i < d; i += 32) { float t = xr[i] - mean; v += t * t; }
  const float rstd = 1.0f / sqrtf(warp_sum(v) / (float)d + eps);
  T* yr = y + (long long)row * d;
  for (int i = lane; i < d; i += 32) yr[i] = from_f<T>((xr[i] - mean) * rstd * g[i] + bta[i]);
}

}  // namespace vadusa
