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
#pragma once
#include "tc.cuh"

namespace vadusa {

constexpr int kGemmBK = 64;                 // K elements per stage (128 bytes per row: one swizzle row)
constexpr int kGemmRowsW = 128;             // weight rows per tile
constexpr int kGemmSmemBudget = 196 * 1024;

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

template <int TN, typename Epi>
__global__ void __launch_bounds__(128) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW,
                                                      const __grid_constant__ CUtensorMap tmX, int M, int N,
                                                      int chunks_per_split, int ksplit, int S, int ring_bytes,
                                                      Epi epi, float* __restrict__ part /*split-K exchange*/, uint32_t* err) {
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
      mbar_expect_tx(full0 + 8 * i, kWBytes + kXBytes);
      tma_load_3d(base + i * Cfg::kStageBytes, &tmW, full0 + 8 * i, (chunk0 + i) * kGemmBK, n0, zb);
    }
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
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = umma_idesc_bf16(kGemmRowsW, TN < 16 ? 16 : TN);
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
      const float* a = part + tile_id * (TN * kGemmRowsW) + t * kGemmRowsW + n4;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float4 pv[8];
#pragma unroll
      for (int peer = 0; peer < 8; ++peer)
        if (peer < ksplit) pv[peer] = __ldcg(reinterpret_cast<const float4*>(a + (long long)peer * (TN * kGemmRowsW)));
#pragma unroll
      for (int peer = 0; peer < 8; ++peer)
        if (peer < ksplit) { acc.x += pv[peer].x; acc.y += pv[peer].y; acc.z += pv[peer].z; acc.w += pv[peer].w; }
      if (m0 + t < M && n0 + n4 < N) epi.vec4(zb, m0 + t, n0 + n4, acc);     // N is a multiple of 4
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace vadusa
