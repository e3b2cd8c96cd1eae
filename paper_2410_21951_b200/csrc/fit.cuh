// Fitting of the draft heads with the base model frozen (paper Sec. II-A: the i-th draft head is supervised by
// a cross-entropy loss multiplied by lambda^i; Sec. III-A.2: heads trained with a fixed base model).  Not on
// the decoding path: plain fp32 FMA kernels on fp32 master copies of the heads; after every step the heads in
// the weight blob are rewritten in the model dtype.
#pragma once
#include "common.cuh"

namespace vadusa {

// C[z][m][n] = sum_k A[z][m * sam + k * sak] * B[z][n * sbn + k * sbk]   (fp32, any strides: the same kernel
// serves X W^T, X^T Y and X W).  64 x 64 tile, K step 16, 256 threads, 4 x 4 outputs per thread.
__global__ void __launch_bounds__(256) fit_gemm_kernel(const float* __restrict__ A, const float* __restrict__ B,
                                                       float* __restrict__ C, int M, int N, int K, long long sam,
                                                       long long sak, long long sbn, long long sbk, long long ldc,
                                                       long long az, long long bz, long long cz) {
  __shared__ float As[16][64 + 4];
  __shared__ float Bs[16][64 + 4];
  A += blockIdx.z * az; B += blockIdx.z * bz; C += blockIdx.z * cz;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
    // 1024 elements of each operand tile, 4 per thread; consecutive threads along the unit-stride axis
    for (int e = threadIdx.x; e < 1024; e += 256) {
      int r, k;
      if (sak == 1) { k = e & 15; r = e >> 4; } else { r = e & 63; k = e >> 6; }
      As[k][r] = (m0 + r < M && k0 + k < K) ? A[(long long)(m0 + r) * sam + (long long)(k0 + k) * sak] : 0.f;
      if (sbk == 1) { k = e & 15; r = e >> 4; } else { r = e & 63; k = e >> 6; }
      Bs[k][r] = (n0 + r < N && k0 + k < K) ? B[(long long)(n0 + r) * sbn + (long long)(k0 + k) * sbk] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; b[i] = Bs[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < M && n < N) C[(long long)m * ldc + n] = acc[i][j];
    }
}

template <typename T>
__global__ void fit_to_f32_kernel(const T* __restrict__ src, float* __restrict__ dst, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = to_f<T>(src[i]);
}

// pre <- pre + b (kept for the backward pass); z = h + SiLU(pre).  grid.y = head.
__global__ void fit_hidden_kernel(float* __restrict__ pre, const float* __restrict__ b, const float* __restrict__ h,
                                  float* __restrict__ z, int T, int d, long long head_stride) {
  const int head = blockIdx.y;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)T * d) return;
  const int col = (int)(i % d);
  const float t = pre[head * head_stride + i] + b[head * d + col];
  pre[head * head_stride + i] = t;
  z[head * head_stride + i] = h[i] + t / (1.0f + expf(-t));
}

// Targets per head that are >= 0.  One block.
__global__ void fit_count_kernel(const int32_t* __restrict__ targets, int T, int heads, int32_t* __restrict__ count) {
  __shared__ int s[32];
  for (int hd = 0; hd < heads; ++hd) {
    int c = 0;
    for (int t = threadIdx.x; t < T; t += blockDim.x) c += targets[(long long)t * heads + hd] >= 0 ? 1 : 0;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += s[w];
      count[hd] = tot;
    }
  }
}

// One block per (position, head): softmax of the logits row over the vocabulary, the row's cross-entropy, and the
// row of d loss / d logits = lambda^(head+1) / count * (p - onehot) written over the logits (zero for a position
// without a target and in the padding columns).
__global__ void __launch_bounds__(256) fit_softmax_ce_kernel(float* __restrict__ logits, const int32_t* __restrict__ targets,
                                                             const int32_t* __restrict__ count, int T, int heads, int vocab,
                                                             int ld, float lambda, float* __restrict__ ce) {
  __shared__ float red[32];
  const int t = blockIdx.x, head = blockIdx.y;
  float* row = logits + ((long long)head * T + t) * ld;
  const int tg = targets[(long long)t * heads + head];
  auto block_reduce = [&](float v, bool is_max) -> float {
    for (int o = 16; o > 0; o >>= 1) {
      const float u = __shfl_xor_sync(0xffffffffu, v, o);
      v = is_max ? fmaxf(v, u) : v + u;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = is_max ? -INFINITY : 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r = is_max ? fmaxf(r, red[w]) : r + red[w];
    return r;
  };
  if (tg < 0 || tg >= vocab) {
    for (int j = threadIdx.x; j < ld; j += blockDim.x) row[j] = 0.f;
    if (threadIdx.x == 0) ce[(long long)head * T + t] = 0.f;
    return;
  }
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x) mx = fmaxf(mx, row[j]);
  mx = block_reduce(mx, true);
  float sum = 0.f;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x) sum += expf(row[j] - mx);
  sum = block_reduce(sum, false);
  float w = 1.0f;
  for (int i = 0; i <= head; ++i) w *= lambda;
  w /= (float)count[head];
  const float inv = 1.0f / sum;
  if (threadIdx.x == 0) ce[(long long)head * T + t] = logf(sum) + mx - row[tg];
  __syncthreads();
  for (int j = threadIdx.x; j < ld; j += blockDim.x) {
    float g = 0.f;
    if (j < vocab) g = w * (expf(row[j] - mx) * inv - (j == tg ? 1.0f : 0.0f));
    row[j] = g;
  }
}

// loss[1 + head] = mean cross-entropy of the head over its targets; loss[0] = sum_i lambda^(i+1) loss[1 + i].  One block,
// fixed summation order.
__global__ void fit_loss_kernel(const float* __restrict__ ce, const int32_t* __restrict__ count, int T, int heads,
                                float lambda, float* __restrict__ loss) {
  __shared__ float red[32];
  float total = 0.f, w = 1.f;
  for (int hd = 0; hd < heads; ++hd) {
    float s = 0.f;
    for (int t = threadIdx.x; t < T; t += blockDim.x) s += ce[(long long)hd * T + t];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    float tot = 0.f;
    for (int q = 0; q < (int)(blockDim.x >> 5); ++q) tot += red[q];
    const float mean = count[hd] > 0 ? tot / (float)count[hd] : 0.f;
    w *= lambda;
    total += w * mean;
    if (threadIdx.x == 0 && loss) loss[1 + hd] = mean;
  }
  if (threadIdx.x == 0 && loss) loss[0] = total;
}

// dpre = dz * SiLU'(pre) in place over dz.  grid.y = head.
__global__ void fit_dpre_kernel(float* __restrict__ dz, const float* __restrict__ pre, long long n, long long head_stride) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const long long o = blockIdx.y * head_stride + i;
  const float t = pre[o], s = 1.0f / (1.0f + expf(-t));
  dz[o] *= s * (1.0f + t * (1.0f - s));
}

// db[head][j] = sum_t dpre[head][t][j].  grid = (ceil(d / 256), heads).
__global__ void fit_colsum_kernel(const float* __restrict__ dpre, float* __restrict__ db, int T, int d, long long head_stride) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x, head = blockIdx.y;
  if (j >= d) return;
  float s = 0.f;
  for (int t = 0; t < T; ++t) s += dpre[head * head_stride + (long long)t * d + j];
  db[head * d + j] = s;
}

// Adam on n parameters; the updated value also goes, in the model dtype, to `deployed` (the weight blob).
template <typename T>
__global__ void fit_adam_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
                                T* __restrict__ deployed, long long n, float lr, float c1, float c2 /*1 - beta^t*/) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float gi = g[i];
  const float mi = 0.9f * m[i] + 0.1f * gi;
  const float vi = 0.999f * v[i] + 0.001f * gi * gi;
  m[i] = mi; v[i] = vi;
  const float np_ = p[i] - lr * (mi / c1) / (sqrtf(vi / c2) + 1e-8f);
  p[i] = np_;
  deployed[i] = from_f<T>(np_);
}

}  // namespace vadusa
