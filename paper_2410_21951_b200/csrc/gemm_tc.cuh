// bf16 projections on the 5th-generation tensor cores (tcgen05.mma, TMEM accumulator,
// TMA-staged operands):  C[m, n] = sum_k X[m, k] * W[n, k], fp32 accumulation.
//
// The weight tile is the MMA's 128-row operand (A) and the token tile its narrow operand
// (B, TN = 16..256 tokens), so with few tokens (batch 1: 64 tree nodes) a CTA still streams
// a full 128 x 64 weight tile per MMA group and the kernel is bound by weight streaming.
// The accumulator D[128 features][TN tokens] lives in tensor memory: lane = feature.
//
// Work split: grid.x = feature tiles of 128, grid.y = token tiles of TN, grid.z = batch *
// ksplit.  With ksplit > 1 the CTAs of one cluster (1,1,ksplit) each take a K slice, park
// their partial tile in an exchange area in global memory (it stays in L2, which moves these
// tiles faster than distributed shared memory did), meet at a cluster barrier, and add the
// slices in a fixed order (deterministic), each CTA finishing TN/ksplit tokens of the tile.
//
// Warp roles (128 threads): warp 0 lane 0 issues TMA loads into a ring of stages, warp 1
// owns the TMEM allocation and its lane 0 issues the MMAs, all four warps run the epilogue.
// Weight tiles of the first stages are requested before griddepcontrol.wait, so under
// programmatic dependent launch they stream while the producer of X is still running.
//
// LN variant (few tokens, one token tile, K slices of 128 columns): X is not read by TMA but
// made in the kernel as LayerNorm(x) of the fp32 residual stream.  The kernel that last wrote
// x (a residual product) left, per row and per group of 128 features, the mean and the sum of
// squared deviations; they are combined exactly (Chan's formula for equal group sizes, fixed
// order), and the normalised, scaled and shifted slice is written as bf16 straight into the
// operand's swizzled shared-memory layout.
#pragma once
#include "tc.cuh"

namespace vadusa {

constexpr int kGemmBK = 64;                 // K elements per stage (128 bytes per row: one swizzle row)
constexpr int kGemmRowsW = 128;             // weight rows per tile
constexpr int kGemmSmemBudget = 196 * 1024;
constexpr int kGemmMaxSplit = 16;           // K slices per tile = cluster size (above 8: non-portable cluster size)

template <int TN> struct GemmTcCfg {
  static constexpr int kStageBytes = kGemmRowsW * kGemmBK * 2 + TN * kGemmBK * 2;
  // wide token tiles (tensor-bound shapes): half the budget per CTA, so that two CTAs share an SM and one's
  // epilogue overlaps the other's main loop; narrow tiles (weight streaming): the whole budget, up to 8 stages
  static constexpr int kStagesMax = (TN >= 128 ? kGemmSmemBudget / 2 : kGemmSmemBudget) / kStageBytes;
  static constexpr int kStages = kStagesMax > 8 ? 8 : kStagesMax;
  static constexpr int kTmemCols = TN < 32 ? 32 : TN;
  // Shared memory needed for `chunks` K chunks per CTA: no more stages than chunks (so that
  // several CTAs fit on an SM).
  static int stages_for(int chunks) { return chunks < kStages ? chunks : kStages; }
  static int ring_for(int chunks, int) { return stages_for(chunks) * kStageBytes; }
  static int smem_for(int chunks, int ksplit) { return ring_for(chunks, ksplit) + 1024 /*alignment*/ + 256 /*barriers*/; }
  static constexpr int kSmemMax = kStages * kStageBytes + 1024 + 256;
};

// LayerNorm fused into the operand load (LN variant).
struct LnFuse {
  const float* x;        // [M][ld] fp32 rows to normalise
  const float* g;        // [K] gain
  const float* b;        // [K] shift
  const float2* stats;   // [M][K/128] (mean, sum of squared deviations) of each group of 128 features
  bf16* y;               // if not null: the CTAs of feature tile 0 also store the normalised rows here ([M][ld] bf16)
  int ld;
  float eps;
};

// All 128 threads; warp w owns rows [w*TN/4, (w+1)*TN/4) of the token tile.  The K slice is the
// 128 columns starting at k0 (two operand tiles of 64 columns); lane l holds columns 4l .. 4l+3.
// K / 128 <= 8 groups per row.
template <int TN>
__device__ __forceinline__ void ln_operand(const LnFuse& ln, int M, int K, int k0, uint32_t x_stage0, uint32_t stage_bytes) {
  constexpr int RPW = TN / 4;                      // rows per warp (multiple of 4)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = K >> 7;
  // gain and shift are weights: fetched while the producer of x is still running
  const float4 gg = __ldg(reinterpret_cast<const float4*>(ln.g + k0 + 4 * lane));
  const float4 bb = __ldg(reinterpret_cast<const float4*>(ln.b + k0 + 4 * lane));
  grid_dep_wait();
  // every load that depends on the producer is issued before the first use: one round trip
  float4 v[RPW];
  float2 st[RPW / 4];
  const int rr = lane >> 3, t = lane & 7;
#pragma unroll
  for (int it = 0; it < RPW / 4; ++it) {
    const int row = warp * RPW + 4 * it + rr;
    st[it] = (t < nt && row < M) ? __ldcg(ln.stats + (long long)row * nt + t) : make_float2(0.f, 0.f);
  }
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    const int row = warp * RPW + r;
    v[r] = row < M ? __ldcg(reinterpret_cast<const float4*>(ln.x + (long long)row * ln.ld + k0 + 4 * lane))
                   : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  // row statistics from the groups': lane = 8 * (row in a group of four rows) + feature group
  float mean_g[RPW / 4], rstd_g[RPW / 4];
  const float inv_nt = 1.0f / (float)nt, inv_k = 1.0f / (float)K;     // (exact for the usual powers of two)
  {
#pragma unroll
    for (int it = 0; it < RPW / 4; ++it) {
      float m = st[it].x;
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
      m *= inv_nt;
      const float dv = st[it].x - m;
      float m2 = t < nt ? st[it].y + 128.0f * dv * dv : 0.f;
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) m2 += __shfl_xor_sync(0xffffffffu, m2, o);
      mean_g[it] = m;
      rstd_g[it] = rsqrtf(fmaf(m2, inv_k, ln.eps));
    }
  }
  // normalise into the swizzled K-major operand tiles: column 4*lane is in tile lane/16, 16-byte unit
  // (lane%16)/2 of the row (xor row%8), half lane&1
  const uint32_t tile = x_stage0 + (uint32_t)(lane >> 4) * stage_bytes + (uint32_t)(lane & 1) * 8u;
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    const int row = warp * RPW + r;
    const float m = __shfl_sync(0xffffffffu, mean_g[r / 4], 8 * (r % 4));
    const float rs = __shfl_sync(0xffffffffu, rstd_g[r / 4], 8 * (r % 4));
    uint32_t lo = 0u, hi = 0u;
    if (row < M) {
      const __nv_bfloat162 p0 = __floats2bfloat162_rn((v[r].x - m) * rs * gg.x + bb.x, (v[r].y - m) * rs * gg.y + bb.y);
      const __nv_bfloat162 p1 = __floats2bfloat162_rn((v[r].z - m) * rs * gg.z + bb.z, (v[r].w - m) * rs * gg.w + bb.w);
      lo = *reinterpret_cast<const uint32_t*>(&p0);
      hi = *reinterpret_cast<const uint32_t*>(&p1);
    }
    const uint32_t unit = (uint32_t)((lane & 15) >> 1) ^ (uint32_t)(row & 7);
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(tile + (uint32_t)row * 128u + (unit << 4)), "r"(lo), "r"(hi));
    if (ln.y != nullptr && blockIdx.x == 0 && row < M)
      *reinterpret_cast<uint2*>(ln.y + (long long)row * ln.ld + k0 + 4 * lane) = make_uint2(lo, hi);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tensor-core reads
}

template <int TN, typename Epi, bool LN = false>
__global__ void __launch_bounds__(128) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW,
                                                      const __grid_constant__ CUtensorMap tmX, int M, int N,
                                                      int chunks_per_split, int ksplit, int S, int ring_bytes,
                                                      Epi epi, float* __restrict__ part /*split-K exchange*/, uint32_t* err,
                                                      LnFuse ln = LnFuse{}) {
  using Cfg = GemmTcCfg<TN>;
  constexpr uint32_t kWBytes = kGemmRowsW * kGemmBK * 2, kXBytes = TN * kGemmBK * 2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + ring_bytes;               // full[S], empty[S], accum, tmem holder
  const uint32_t full0 = bars, empty0 = bars + 8 * S, accum_bar = bars + 16 * S, holder = bars + 16 * S + 8;
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(ring_ptr + ring_bytes + 16 * S + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kGemmRowsW, m0 = blockIdx.y * TN;
  const int zb = blockIdx.z / ksplit, ks = blockIdx.z % ksplit;
  const int chunk0 = ks * chunks_per_split, nchunks = chunks_per_split;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(accum_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmX);
  }
  if (warp == 1) { tmem_alloc(holder, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;
  if (warp == 0 && lane == 0) {
    // ---- TMA producer
    const int pre = nchunks < S ? nchunks : S;
    for (int i = 0; i < pre; ++i) {                      // weights do not depend on the upstream kernel
      mbar_expect_tx(full0 + 8 * i, LN ? kWBytes : kWBytes + kXBytes);
      tma_load_3d(base + i * Cfg::kStageBytes, &tmW, full0 + 8 * i, (chunk0 + i) * kGemmBK, n0, zb);
    }
    if constexpr (!LN) {
      grid_dep_wait();
      for (int i = 0; i < pre; ++i)
        tma_load_3d(base + i * Cfg::kStageBytes + kWBytes, &tmX, full0 + 8 * i, (chunk0 + i) * kGemmBK, m0, zb);
      for (int i = pre; i < nchunks; ++i) {
        const int s = i % S;
        if (!mbar_wait(empty0 + 8 * s, ((i / S) - 1) & 1, err)) break;
        mbar_expect_tx(full0 + 8 * s, kWBytes + kXBytes);
        tma_load_3d(base + s * Cfg::kStageBytes, &tmW, full0 + 8 * s, (chunk0 + i) * kGemmBK, n0, zb);
        tma_load_3d(base + s * Cfg::kStageBytes + kWBytes, &tmX, full0 + 8 * s, (chunk0 + i) * kGemmBK, m0, zb);
      }
    }
  }
  if constexpr (LN) {
    // every chunk of the slice has a stage of its own (nchunks <= S): all threads build the X tiles
    __syncwarp();
    if constexpr (TN <= 64)                          // (waits for the producer of x inside)
      ln_operand<TN>(ln, M, nchunks * ksplit * kGemmBK, chunk0 * kGemmBK, base + kWBytes, Cfg::kStageBytes);
    __syncthreads();
  }
  if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = umma_idesc_bf16(kGemmRowsW, TN < 16 ? 16 : TN);
    // the token operand is requested only after the upstream grid has finished: wait for that first, so that the
    // bounded waits below time this kernel's own pipeline and not the upstream kernel's run time
    grid_dep_wait();
    for (int i = 0; i < nchunks; ++i) {
      const int s = i % S;
      if (!mbar_wait(full0 + 8 * s, (i / S) & 1, err)) break;
      tc_fence_after();
      const uint32_t wa = base + s * Cfg::kStageBytes, xa = wa + kWBytes;
#pragma unroll
      for (int k = 0; k < kGemmBK / 16; ++k)
        umma_bf16(tmem, umma_desc_k_sw128(wa + 32 * k), umma_desc_k_sw128(xa + 32 * k), idesc, (i | k) != 0);
      umma_commit(empty0 + 8 * s);                       // stage reusable once these MMAs have read it
    }
    umma_commit(accum_bar);                              // accumulator complete
  }
  __syncwarp();
  // every thread (grid_dep_wait must precede any global access of upstream-produced data)
  grid_dep_wait();
  mbar_wait(accum_bar, 0, err);
  tc_fence_after();
  grid_dep_launch();

  // ---- epilogue: warp w reads TMEM lanes 32w .. 32w+31 (features n0 + 32w + lane)
  const int n = n0 + 32 * warp + lane;
  const uint32_t trow = tmem + ((uint32_t)(32 * warp) << 16);
  if (ksplit == 1) {
    constexpr int CH = TN < 32 ? 16 : 32;
#pragma unroll 1
    for (int c0 = 0; c0 < TN; c0 += CH) {
      float v[CH];
      if (CH == 32) tmem_ld32(trow + c0, v); else tmem_ld16(trow + c0, v);
      if (n < N && m0 + c0 < M) epi.template col<CH>(zb, m0 + c0, n, v, M - (m0 + c0));
    }
  } else {
    // park the partial tile as P[token][feature] in the exchange area of this (tile, slice); the slices of
    // a tile are summed in a fixed order, CTA ks finishing tokens [ks*per, (ks+1)*per)
    const long long tile_id = ((long long)blockIdx.x * gridDim.y + blockIdx.y) * gridDim.z + (long long)zb * ksplit;
    float* P = part + (tile_id + ks) * (TN * kGemmRowsW);
    constexpr int CH = TN < 32 ? 16 : 32;
#pragma unroll 1
    for (int c0 = 0; c0 < TN; c0 += CH) {
      float v[CH];
      if (CH == 32) tmem_ld32(trow + c0, v); else tmem_ld16(trow + c0, v);
#pragma unroll
      for (int j = 0; j < CH; ++j) P[(c0 + j) * kGemmRowsW + threadIdx.x] = v[j];
    }
    cluster_sync_all();                                  // release / acquire: the peers' tiles are visible
    const int per = TN / ksplit;
    const int n4 = (threadIdx.x & 31) * 4;
    for (int t = ks * per + warp; t < (ks + 1) * per; t += 4) {
      // (one block, so that the epilogue's own loads can be issued beside the peers')
      if (m0 + t < M && n0 + n4 < N) {                                        // N is a multiple of 4
        const float* a = part + tile_id * (TN * kGemmRowsW) + t * kGemmRowsW + n4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float4 pv[kGemmMaxSplit];
#pragma unroll
        for (int peer = 0; peer < kGemmMaxSplit; ++peer)
          if (peer < ksplit) pv[peer] = __ldcg(reinterpret_cast<const float4*>(a + (long long)peer * (TN * kGemmRowsW)));
#pragma unroll
        for (int peer = 0; peer < kGemmMaxSplit; ++peer)
          if (peer < ksplit) { acc.x += pv[peer].x; acc.y += pv[peer].y; acc.z += pv[peer].z; acc.w += pv[peer].w; }
        epi.vec4(zb, m0 + t, n0 + n4, acc);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace vadusa
