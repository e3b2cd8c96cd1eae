// Plain FMA matrix product C[m,n] = sum_k A[m,k] * W[n,k] with fused epilogues.
// This is the arithmetic of the fp32 model type (no tensor-core rounding); the
// bf16 model type uses the tensor-core kernels and only falls back to this
// file for shapes those do not cover.
#pragma once
#include "common.cuh"

namespace vadusa {

// ---- epilogues: called with the fp32 accumulator, one element at a time (operator()) or
// four consecutive features of one token at a time (vec4; n is a multiple of 4) ----------

// q/k/v projection (verify step, per layer): + bias, round to T; q goes to a dense buffer,
// k and v go straight to the paged cache at the node's slot (kv_row[m], written by the
// embedding kernel of the same pass; -1: the row is not scored).
template <typename T>
struct EpiQKV {
  const float* bias;
  T* q;
  T* pool;                      // KV pool of this layer
  const long long* kv_row;      // [M] element offset of the row's K slot for head 0
  long long kv_stride;          // elements from a K row to the V row of the same head
  int tile_elems;               // elements between heads: 64 * head_dim
  int head_dim, d;
  __device__ __forceinline__ long long kv_elem(long long row, int n) const {
    const int c = n - d, kv = c >= d, cc = c - kv * d, h = cc / head_dim;
    return row + kv * kv_stride + (long long)h * tile_elems + (cc - h * head_dim);
  }
  __device__ __forceinline__ void operator()(int, int m, int n, float acc) const {
    const T r = from_f<T>(acc + bias[n]);
    if (n < d) { q[(long long)m * d + n] = r; return; }
    const long long row = kv_row[m];
    if (row >= 0) pool[kv_elem(row, n)] = r;
  }
  __device__ __forceinline__ void vec4(int, int m, int n, float4 a) const {
    const float4 b = *reinterpret_cast<const float4*>(bias + n);
    if (n < d) { store4<T>(q + (long long)m * d + n, a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); return; }
    const long long row = kv_row[m];
    if (row >= 0) store4<T>(pool + kv_elem(row, n), a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
  }
  // CH consecutive tokens m .. m+count-1 of one feature n (all loads first, then the stores)
  template <int CH>
  __device__ __forceinline__ void col(int, int m, int n, const float* v, int count) const {
    const float b = bias[n];
    if (n < d) {
#pragma unroll
      for (int j = 0; j < CH; ++j)
        if (j < count) q[(long long)(m + j) * d + n] = from_f<T>(v[j] + b);
      return;
    }
    long long rows[CH];
#pragma unroll
    for (int j = 0; j < CH; ++j) rows[j] = j < count ? kv_row[m + j] : -1;
    const long long off = kv_elem(0, n);
#pragma unroll
    for (int j = 0; j < CH; ++j)
      if (rows[j] >= 0) pool[rows[j] + off] = from_f<T>(v[j] + b);
  }
};

// output projection / second feed-forward matrix: x += acc + bias (fp32 residual stream)
struct EpiResidual {
  const float* bias;
  float* x;
  int ld;
  __device__ __forceinline__ void operator()(int, int m, int n, float acc) const {
    x[(long long)m * ld + n] += acc + bias[n];
  }
  __device__ __forceinline__ void vec4(int, int m, int n, float4 a) const {
    const float4 b = *reinterpret_cast<const float4*>(bias + n);
    float4* p = reinterpret_cast<float4*>(x + (long long)m * ld + n);
    float4 v = *p;
    v.x += a.x + b.x; v.y += a.y + b.y; v.z += a.z + b.z; v.w += a.w + b.w;
    *p = v;
  }
  template <int CH>
  __device__ __forceinline__ void col(int, int m, int n, const float* v, int count) const {
    const float b = bias[n];
    float xv[CH];
#pragma unroll
    for (int j = 0; j < CH; ++j) xv[j] = j < count ? x[(long long)(m + j) * ld + n] : 0.f;
#pragma unroll
    for (int j = 0; j < CH; ++j)
      if (j < count) x[(long long)(m + j) * ld + n] = xv[j] + (v[j] + b);
  }
};

// EpiResidual that also leaves, per row and group of 128 features, the mean and the sum of squared
// deviations of the updated residual stream (the LayerNorm-fused product reads them).  vec4 must be
// called by all 32 lanes of a warp with the same row m and n = (a multiple of 128) + 4 * lane.
struct EpiResidualStats {
  const float* bias;
  float* x;
  int ld;
  float2* stats;          // [rows][ld / 128]
  __device__ __forceinline__ void operator()(int, int m, int n, float acc) const {
    x[(long long)m * ld + n] += acc + bias[n];
  }
  __device__ __forceinline__ void vec4(int, int m, int n, float4 a) const {
    const float4 b = *reinterpret_cast<const float4*>(bias + n);
    float4* p = reinterpret_cast<float4*>(x + (long long)m * ld + n);
    float4 v = *p;
    v.x += a.x + b.x; v.y += a.y + b.y; v.z += a.z + b.z; v.w += a.w + b.w;
    *p = v;
    float s = (v.x + v.y) + (v.z + v.w);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mu = s * (1.0f / 128.0f);
    const float d0 = v.x - mu, d1 = v.y - mu, d2 = v.z - mu, d3 = v.w - mu;
    float q = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    if ((threadIdx.x & 31) == 0) stats[(long long)m * (ld >> 7) + (n >> 7)] = make_float2(mu, q);
  }
  template <int CH>
  __device__ __forceinline__ void col(int z, int m, int n, const float* v, int count) const {
    EpiResidual{bias, x, ld}.template col<CH>(z, m, n, v, count);     // no statistics on this path
  }
};

// first feed-forward matrix: relu(acc + bias) rounded to T
template <typename T>
struct EpiRelu {
  const float* bias;
  T* out;
  int ld;
  __device__ __forceinline__ void operator()(int, int m, int n, float acc) const {
    out[(long long)m * ld + n] = from_f<T>(fmaxf(acc + bias[n], 0.f));
  }
  __device__ __forceinline__ void vec4(int, int m, int n, float4 a) const {
    const float4 b = *reinterpret_cast<const float4*>(bias + n);
    store4<T>(out + (long long)m * ld + n, fmaxf(a.x + b.x, 0.f), fmaxf(a.y + b.y, 0.f), fmaxf(a.z + b.z, 0.f),
              fmaxf(a.w + b.w, 0.f));
  }
  template <int CH>
  __device__ __forceinline__ void col(int, int m, int n, const float* v, int count) const {
    const float b = bias[n];
#pragma unroll
    for (int j = 0; j < CH; ++j)
      if (j < count) out[(long long)(m + j) * ld + n] = from_f<T>(fmaxf(v[j] + b, 0.f));
  }
};

// vocabulary heads: fp32 logits; z selects the draft head
struct EpiLogits {
  float* out;
  int ld;
  long long z_stride;
  __device__ __forceinline__ void operator()(int z, int m, int n, float acc) const {
    out[z * z_stride + (long long)m * ld + n] = acc;
  }
  __device__ __forceinline__ void vec4(int z, int m, int n, float4 a) const {
    *reinterpret_cast<float4*>(out + z * z_stride + (long long)m * ld + n) = a;
  }
  template <int CH>
  __device__ __forceinline__ void col(int z, int m, int n, const float* v, int count) const {
#pragma unroll
    for (int j = 0; j < CH; ++j)
      if (j < count) out[z * z_stride + (long long)(m + j) * ld + n] = v[j];
  }
};

// draft residual block (Sec. III-A.1): z = h + SiLU(acc + bias), rounded to T; z selects the head
template <typename T>
struct EpiDraftHidden {
  const float* bias;     // [heads][d]
  const T* h;            // [batch][d]
  T* out;                // [heads][batch][d]
  int d, batch;
  __device__ __forceinline__ void operator()(int z, int m, int n, float acc) const {
    const float t = acc + bias[z * d + n];
    const float s = t / (1.0f + expf(-t));
    out[((long long)z * batch + m) * d + n] = from_f<T>(to_f<T>(h[(long long)m * d + n]) + s);
  }
};

// the same with the heads' matrices stacked along the feature axis: n = head * d + column
template <typename T>
struct EpiDraftHiddenFlat {
  const float* bias;     // [heads * d]
  const T* h;            // [batch][d]
  T* out;                // [heads][batch][d]
  int d, batch;
  __device__ __forceinline__ void operator()(int, int m, int n, float acc) const {
    const int head = n / d, col = n - head * d;
    const float t = acc + bias[n];
    const float s = t / (1.0f + expf(-t));
    out[((long long)head * batch + m) * d + col] = from_f<T>(to_f<T>(h[(long long)m * d + col]) + s);
  }
  __device__ __forceinline__ void vec4(int z, int m, int n, float4 a) const {
    (*this)(z, m, n, a.x); (*this)(z, m, n + 1, a.y); (*this)(z, m, n + 2, a.z); (*this)(z, m, n + 3, a.w);
  }
  template <int CH>
  __device__ __forceinline__ void col(int z, int m, int n, const float* v, int count) const {
#pragma unroll
    for (int j = 0; j < CH; ++j)
      if (j < count) (*this)(z, m + j, n, v[j]);
  }
};

// ---- kernel -----------------------------------------------------------------------
// 64x64 tile, K step 16, 256 threads, 4x4 outputs per thread.  K must be a multiple of 16.
// grid = (ceil(N/64), ceil(M/64), batches); A and W advance by a_z / w_z elements per batch.
template <typename T, typename Epi>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ W,
                                                        int M, int N, int K, long long a_z, long long w_z, Epi epi) {
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const int z = blockIdx.z;
  A += z * a_z; W += z * w_z;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int lr = threadIdx.x >> 2, lk = (threadIdx.x & 3) * 4;   // loader: row 0..63, k offset 0,4,8,12
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
    {
      const int gm = m0 + lr, gn = n0 + lr;
      float a[4] = {0.f, 0.f, 0.f, 0.f}, w[4] = {0.f, 0.f, 0.f, 0.f};
      if (gm < M) {
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = to_f<T>(A[(long long)gm * K + k0 + lk + i]);
      }
      if (gn < N) {
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = to_f<T>(W[(long long)gn * K + k0 + lk + i]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) { As[lk + i][lr] = a[i]; Ws[lk + i][lr] = w[i]; }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < N) epi(z, m, n, acc[i][j]);
    }
  }
}

}  // namespace vadusa
