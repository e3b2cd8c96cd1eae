// Shared device helpers of libvadusa (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace vadusa {

typedef __nv_bfloat16 bf16;

constexpr int kKvBlock = 64;         // tokens per KV block
constexpr int kMaxNodes = 128;       // two 64-bit ancestor words per node
constexpr int kMaxPath = 16;         // longest root path
constexpr int kStatDepth = 15;       // acceptance statistics: draft heads x top-k ranks (the C ABI's maxima)
constexpr int kStatTopk = 16;
constexpr int kMaxTopk = 16;

// bits of the device error word
enum : uint32_t {
  kErrCapacity = 1u,   // a block-table entry or position was out of range
  kErrTimeout = 2u     // a bounded wait expired
};

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// value after the storage rounding of the model dtype
template <typename T> __device__ __forceinline__ float round_as(float v) { return to_f<T>(from_f<T>(v)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Total order used for every integer decision: larger value first, then lower id.
__device__ __forceinline__ bool precedes(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}

// Geometry of the paged KV pool of one layer: [block][2][head][64][head_dim].
struct KvGeom {
  int n_heads, head_dim, max_blocks_per_seq;
  long long num_blocks;
  long long layer_stride;   // elements between layers
  __device__ __forceinline__ long long elem(long long blk, int kv, int h, int off) const {
    return (((blk * 2 + kv) * n_heads + h) * (long long)kKvBlock + off) * head_dim;
  }
};

// Block id of logical position pos of sequence b, or -1 (and the error bit) if the
// table does not cover it.  Every dereference of the block table goes through here.
__device__ __forceinline__ long long kv_block_of(const int32_t* __restrict__ block_table, const KvGeom& g,
                                                 int b, int pos, uint32_t* err) {
  int pi = pos / kKvBlock;
  if (pos < 0 || pi >= g.max_blocks_per_seq) { atomicOr(err, kErrCapacity); return -1; }
  long long blk = block_table[(long long)b * g.max_blocks_per_seq + pi];
  if (blk < 0 || blk >= g.num_blocks) { atomicOr(err, kErrCapacity); return -1; }
  return blk;
}

// Per-call view of the candidate tree.  Arrays are [n_nodes] (shared) or
// [batch][n_nodes] (per_seq != 0).
struct TreeView {
  const int32_t* parent;
  const int32_t* depth;
  const int32_t* rank;
  const unsigned long long* anc;   // ancestor-or-self bits, two words per node (bits 0..63, 64..127)
  int n_nodes;
  int per_seq;
  __device__ __forceinline__ int off(int b) const { return per_seq ? b * n_nodes : 0; }
  __device__ __forceinline__ void anc_of(int b, int n, unsigned long long& lo, unsigned long long& hi) const {
    const unsigned long long* p = anc + 2ll * (off(b) + n);
    lo = p[0]; hi = p[1];
  }
};

// Bits [rel, rel + 32) of the 128-bit word (hi:lo), rel in [0, 128); bits beyond 127 read as zero.
__device__ __forceinline__ uint32_t bits32_at(unsigned long long lo, unsigned long long hi, int rel) {
  if (rel < 64) {
    uint32_t v = (uint32_t)(lo >> rel);
    if (rel > 32) v |= (uint32_t)(hi << (64 - rel));
    return v;
  }
  return (uint32_t)(hi >> (rel - 64));
}
__device__ __forceinline__ bool bit_at(unsigned long long lo, unsigned long long hi, int i) {
  return ((i < 64 ? lo >> i : hi >> (i - 64)) & 1ull) != 0ull;
}

// Four consecutive values rounded to T and stored as one vector.
template <typename T> __device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<bf16>(bf16* p, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = v;
}

}  // namespace vadusa
