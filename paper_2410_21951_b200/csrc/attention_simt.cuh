// Tree-masked decode attention over the paged KV cache, plain FMA arithmetic.
// Node n of sequence b attends to every cached position < ctx_len[b] and to the tree
// slots ctx_len[b] + m whose bit m is set in anc[n] (its ancestors and itself); tree
// nodes' K/V rows sit in the cache behind the context (paper Sec. II-A, tree attention).
#pragma once
#include "common.cuh"

namespace vadusa {

// grid = (heads, batch), 256 threads; warp w owns nodes w, w+8, ...; online softmax per node.
template <typename T, int DH>
__global__ void __launch_bounds__(256) tree_attention_simt_kernel(
    const T* __restrict__ q, const T* __restrict__ pool, const int32_t* __restrict__ block_table,
    const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ nvalid, TreeView tree, KvGeom geom,
    int d_model, float scale, T* __restrict__ out, uint32_t* err) {
  constexpr int R = DH / 32;
  extern __shared__ float smem[];
  float* Qs = smem;                       // [64][DH]
  float* Ks = Qs + 64 * DH;               // [64][DH+1]
  float* Vs = Ks + 64 * (DH + 1);         // [64][DH]
  float* Ps = Vs + 64 * DH;               // [64][64]
  const int N = tree.n_nodes, ntile = (N + 63) >> 6;
  const int h = blockIdx.x, b = (int)blockIdx.y / ntile, nb = 64 * ((int)blockIdx.y % ntile);   // nodes nb .. nb+63
  const int nv = nvalid[b], S = ctx_len[b];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  for (int i = threadIdx.x; i < 64 * DH; i += 256) {
    const int n = i / DH, e = i % DH;
    Qs[i] = (nb + n < N) ? to_f<T>(q[((long long)b * N + nb + n) * d_model + h * DH + e]) : 0.f;
  }
  float O[8][R], mrun[8], lrun[8];
  unsigned long long alo[8], ahi[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    mrun[i] = -INFINITY; lrun[i] = 0.f;
    const int n = warp + 8 * i;
    alo[i] = ahi[i] = 0ull;
    if (nb + n < nv) tree.anc_of(b, nb + n, alo[i], ahi[i]);
#pragma unroll
    for (int c = 0; c < R; ++c) O[i][c] = 0.f;
  }
  const int total = S + nv;
  for (int t0 = 0; t0 < total; t0 += kKvBlock) {
    __syncthreads();
    const long long blk = kv_block_of(block_table, geom, b, t0, err);
    if (blk < 0) continue;                                   // uniform over the block
    const T* Kg = pool + geom.elem(blk, 0, h, 0);
    const T* Vg = pool + geom.elem(blk, 1, h, 0);
    for (int i = threadIdx.x; i < 64 * DH; i += 256) {
      const int j = i / DH, e = i % DH;
      const bool live = t0 + j < total;                      // slots past the tree hold stale data
      Ks[j * (DH + 1) + e] = live ? to_f<T>(Kg[i]) : 0.f;
      Vs[i] = live ? to_f<T>(Vg[i]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int n = warp + 8 * i;
      if (nb + n >= nv) continue;
      float s[2];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int j = lane + 32 * c, p = t0 + j;
        float a = 0.f;
        for (int e = 0; e < DH; ++e) a = fmaf(Qs[n * DH + e], Ks[j * (DH + 1) + e], a);
        const bool vis = p < S || (p < total && bit_at(alo[i], ahi[i], p - S));
        s[c] = vis ? a * scale : -INFINITY;
      }
      const float mnew = fmaxf(mrun[i], warp_max(fmaxf(s[0], s[1])));
      if (mnew == -INFINITY) continue;
      const float p0 = expf(s[0] - mnew), p1 = expf(s[1] - mnew);
      const float corr = expf(mrun[i] - mnew);
      lrun[i] = lrun[i] * corr + warp_sum(p0 + p1);
      mrun[i] = mnew;
      Ps[n * 64 + lane] = p0;
      Ps[n * 64 + lane + 32] = p1;
#pragma unroll
      for (int c = 0; c < R; ++c) O[i][c] *= corr;
      __syncwarp();
      for (int j = 0; j < 64; ++j) {
        const float pj = Ps[n * 64 + j];
#pragma unroll
        for (int c = 0; c < R; ++c) O[i][c] = fmaf(pj, Vs[j * DH + lane + 32 * c], O[i][c]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int n = warp + 8 * i;
    if (nb + n >= N) continue;
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const float v = (nb + n < nv && lrun[i] > 0.f) ? O[i][c] / lrun[i] : 0.f;
      out[((long long)b * N + nb + n) * d_model + h * DH + lane + 32 * c] = from_f<T>(v);
    }
  }
}

}  // namespace vadusa
