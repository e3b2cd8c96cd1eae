// Position-keyed Gumbel noise and sampling keys (Alg. 1 line 3 realised as Gumbel-top-tau).
#pragma once
#include "common.cuh"

namespace vadusa {

// Output function of splitmix64 (Steele, Lea, Flood 2014).
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;

// Hash state shared by all tokens of one (seed, sequence, predicted position).
__host__ __device__ __forceinline__ uint64_t noise_row_state(uint64_t seed, int seq, int pos) {
  uint64_t a = mix64(seed + kGolden * (uint64_t)(seq + 1));
  return mix64(a + kGolden * (uint64_t)(pos + 1));
}

// g = -log(-log(u)), u = (x + 1/2) / 2^23 with x the top 23 bits of the token's hash.
__device__ __forceinline__ float gumbel_of(uint64_t row_state, int token) {
  uint64_t c = mix64(row_state + kGolden * (uint64_t)(token + 1));
  float u = __fmul_rn((float)(uint32_t)(c >> 41) + 0.5f, 1.1920928955078125e-07f);   // 2^-23
  return -logf(-logf(u));
}

struct SamplingDev {
  int tau;
  float temperature, inv_temperature, top_p;
  int eos_masked, accept_rule, eos_id;
  int bias_ld;                    // row length of bias
  unsigned long long seed;
  const float* bias;              // [batch][bias_ld] added to the base head's logits before anything else, or null
};

// A logits row of the base head as the sampler sees it: logit + bias (one fp32 addition) when a bias is set.
struct BaseRow {
  const float* row;
  const float* bias;
  __device__ __forceinline__ float operator[](int j) const { return bias ? __fadd_rn(row[j], bias[j]) : row[j]; }
};
__device__ __forceinline__ BaseRow base_row(const float* row, const SamplingDev& sp, int seq) {
  return BaseRow{row, sp.bias ? sp.bias + (long long)seq * sp.bias_ld : nullptr};
}

// fp32 key of a token: logit * (1/T) + g, formed with separately rounded operations.
__device__ __forceinline__ float key_of(float logit, int token, uint64_t row_state, const SamplingDev& sp, bool noise) {
  if (sp.eos_masked && token == sp.eos_id) return -INFINITY;
  if (sp.temperature == 0.f || !noise) return logit;
  return __fadd_rn(__fmul_rn(logit, sp.inv_temperature), gumbel_of(row_state, token));
}

// Logit as the sampler sees it (EOS masked).
__device__ __forceinline__ float masked_logit(float logit, int token, const SamplingDev& sp) {
  return (sp.eos_masked && token == sp.eos_id) ? -INFINITY : logit;
}

}  // namespace vadusa
