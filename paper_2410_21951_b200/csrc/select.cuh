// Block-level selection helpers, the root sample and the draft heads' top-k
// (paper Sec. II-A: the base head gives the first next token, draft head i the
// top-k candidates of depth i).
#pragma once
#include "rng.cuh"

namespace vadusa {

struct Best { float v; int i; };

__device__ __forceinline__ Best better(Best a, Best b) {
  if (b.i < 0) return a;
  if (a.i < 0) return b;
  return precedes(a.v, a.i, b.v, b.i) ? a : b;
}

// fp32 -> uint32 that orders like the value (-0 counted as +0); every finite value and -inf map above 0.
__device__ __forceinline__ uint32_t ordered_bits(float v) {
  const uint32_t u = __float_as_uint(__fadd_rn(v, 0.0f));
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// First element of the block in the order "larger value, then lower id" (i < 0: none).
// scratch: 32 Best entries of shared memory.  Result is the same in every thread.  The value travels as
// its ordered bit pattern, so a warp needs two reduction instructions: the largest value, then the lowest
// id among the lanes that hold it.
__device__ __forceinline__ Best block_first(Best x, Best* scratch) {
  const uint32_t none = 0xffffffffu;
  uint32_t k = x.i < 0 ? 0u : ordered_bits(x.v);
  uint32_t wk = __reduce_max_sync(0xffffffffu, k);
  uint32_t wi = __reduce_min_sync(0xffffffffu, (x.i >= 0 && k == wk) ? (uint32_t)x.i : none);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) scratch[warp] = Best{__uint_as_float(wk), (int)wi};
  __syncthreads();
  const bool have = lane < nw && scratch[lane].i != (int)none;
  k = have ? __float_as_uint(scratch[lane].v) : 0u;
  const uint32_t id = have ? (uint32_t)scratch[lane].i : none;
  wk = __reduce_max_sync(0xffffffffu, k);
  wi = __reduce_min_sync(0xffffffffu, (have && k == wk) ? id : none);
  if (wi == none) return Best{0.f, -1};
  return Best{from_ordered_bits(wk), (int)wi};
}

__device__ __forceinline__ float block_sum(float x, float* scratch) {
  x = warp_sum(x);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) scratch[warp] = x;
  __syncthreads();
  float r = (lane < nw) ? scratch[lane] : 0.f;
  return warp_sum(r);
}

__device__ __forceinline__ float block_max(float x, float* scratch) {
  x = warp_max(x);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) scratch[warp] = x;
  __syncthreads();
  float r = (lane < nw) ? scratch[lane] : -INFINITY;
  return warp_max(r);
}

// Softmax statistics of a logits row at the sampling temperature (EOS masked).
struct RowStats { float maxl, z; };

__device__ __forceinline__ RowStats row_stats(const BaseRow row, int vocab, const SamplingDev& sp,
                                              float* scratch) {
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x) mx = fmaxf(mx, masked_logit(row[j], j, sp));
  mx = block_max(mx, scratch);
  float z = 0.f;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x)
    z += expf((masked_logit(row[j], j, sp) - mx) * sp.inv_temperature);
  z = block_sum(z, scratch);
  return RowStats{mx, z};
}

// Nucleus membership of token c (top-p of softmax(logits/T)): the probability mass of the
// tokens ahead of c (larger logit, or equal logit and lower id) is below top_p.
__device__ __forceinline__ bool in_nucleus(const BaseRow row, int vocab, int c, RowStats st,
                                           const SamplingDev& sp, float* scratch) {
  const float lc = masked_logit(row[c], c, sp);
  if (lc == -INFINITY) return false;
  float m = 0.f;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x) {
    const float lj = masked_logit(row[j], j, sp);
    if (precedes(lj, j, lc, c)) m += expf((lj - st.maxl) * sp.inv_temperature);
  }
  m = block_sum(m, scratch);
  return m / st.z < sp.top_p;
}

__device__ __forceinline__ bool nucleus_on(const SamplingDev& sp) {
  return sp.temperature != 0.f && sp.top_p < 1.0f;
}

// The base head's single sample for absolute position pos: the first token, in key order,
// that lies in the nucleus.  Same result in every thread.
__device__ int sample_row(const BaseRow row, int vocab, int seq, int pos, const SamplingDev& sp,
                          Best* bscratch, float* fscratch) {
  const uint64_t rs = noise_row_state(sp.seed, seq, pos);
  const bool nuc = nucleus_on(sp);
  RowStats st{0.f, 1.f};
  if (nuc) st = row_stats(row, vocab, sp, fscratch);
  Best bound{INFINITY, -1};
  for (int tries = 0; tries < vocab; ++tries) {
    Best mine{0.f, -1};
    for (int j = threadIdx.x; j < vocab; j += blockDim.x) {
      const float k = key_of(row[j], j, rs, sp, true);
      if (bound.i >= 0 && !precedes(bound.v, bound.i, k, j)) continue;     // already tried
      mine = better(mine, Best{k, j});
    }
    const Best top = block_first(mine, bscratch);
    if (top.i < 0) break;
    if (!nuc || in_nucleus(row, vocab, top.i, st, sp, fscratch)) return top.i;
    bound = top;
  }
  return 0;
}

// grid = (n_draft_heads + 1, batch).  blockIdx.x < n_draft_heads: the head's top-k ids in
// descending logit order (EOS masked), written to topk[b][head][0..k).  Last x: the root.
__global__ void __launch_bounds__(256) draft_select_kernel(
    const float* __restrict__ dlogits /*[heads][batch][ld]*/, const float* __restrict__ logits_star /*[batch][ld]*/,
    int ld, int vocab, int batch, int n_heads, int k, const int32_t* __restrict__ ctx_len,
    const int32_t* __restrict__ nvalid, SamplingDev sp, int32_t* __restrict__ topk, int32_t* __restrict__ root) {
  __shared__ Best bscratch[32];
  __shared__ float fscratch[32];
  const int b = blockIdx.y, head = blockIdx.x;
  if (nvalid[b] == 0) return;
  if (head == n_heads) {
    const int r = sample_row(base_row(logits_star + (long long)b * ld, sp, b), vocab, b, ctx_len[b], sp, bscratch, fscratch);
    if (threadIdx.x == 0) root[b] = r;
    return;
  }
  const float* row = dlogits + ((long long)head * batch + b) * ld;
  // the row is read once: each thread keeps its first kCache entries in registers (taken ones are
  // struck out there); entries beyond kCache * blockDim.x are re-read and filtered by the last pick
  constexpr int kCache = 8;
  float cv[kCache];
#pragma unroll
  for (int c = 0; c < kCache; ++c) {
    const int j = threadIdx.x + c * blockDim.x;
    cv[c] = j < vocab ? masked_logit(row[j], j, sp) : -INFINITY;
  }
  const int cached = kCache * blockDim.x;
  unsigned taken = 0u;
  Best bound{INFINITY, -1};
  for (int r = 0; r < k; ++r) {
    Best mine{0.f, -1};
#pragma unroll
    for (int c = 0; c < kCache; ++c) {
      const int j = threadIdx.x + c * blockDim.x;
      if (j < vocab && !((taken >> c) & 1u)) mine = better(mine, Best{cv[c], j});
    }
    for (int j = cached + threadIdx.x; j < vocab; j += blockDim.x) {
      const float v = masked_logit(row[j], j, sp);
      if (bound.i >= 0 && !precedes(bound.v, bound.i, v, j)) continue;
      mine = better(mine, Best{v, j});
    }
    const Best top = block_first(mine, bscratch);
    if (threadIdx.x == 0) topk[((long long)b * n_heads + head) * k + r] = top.i < 0 ? 0 : top.i;
#pragma unroll
    for (int c = 0; c < kCache; ++c)
      if (top.i == threadIdx.x + c * blockDim.x) taken |= 1u << c;
    bound = top;
  }
}

}  // namespace vadusa
