// bf16 projections for many tokens (tensor-bound shapes) on CTA pairs: tcgen05.mma.cta_group::2.
// The two CTAs of a cluster compute a 256-feature x TN-token tile together: each CTA stages its own 128
// weight rows (the MMA's A operand) and half of the token tile (TN/2 rows of the B operand); the pair's
// MMA reads both halves of B, so an SM fetches 16 KB + TN/2 * 128 B per 64-wide K step instead of the
// 16 KB + TN * 128 B of the single-CTA kernel: fewer operand bytes from L2 per flop, and a deeper ring in
// the same shared memory.  The accumulator of each CTA (its 128 features x TN tokens) is in its own TMEM.
//
// Protocol: CTA 0 of the pair leads.  Both CTAs issue their TMA loads with the leader's `full` barrier
// as completion barrier (the leader expects the bytes of both); the leader's MMA thread issues the pair's
// MMAs and signals, through tcgen05.commit to both CTAs, the `empty` barrier of a stage and at the
// end the accumulator barrier.  TMEM is allocated and freed by warp 1 of both CTAs; the CTAs
// meet at a cluster barrier after the barrier set-up and before the TMEM is freed.
// No K split and no LayerNorm operand here; every wait is bounded like in the single-CTA kernel.
#pragma once
#include "tc.cuh"
#include "gemm_tc.cuh"

namespace vadusa {

// ST stages of 16 KB of weights + TN/2 token rows.  Several CTAs (of different pairs) share an SM, so that one's
// epilogue overlaps another's main loop: two with <256, 3> (TMEM: 2 x 256 columns) and <128, 4>, three with <128, 3>.
template <int TN, int ST> struct GemmTc2Cfg {
  static constexpr int kXHalfBytes = (TN / 2) * kGemmBK * 2;
  static constexpr int kStageBytes = kGemmRowsW * kGemmBK * 2 + kXHalfBytes;
  static constexpr int kStages = ST;
  static constexpr int kTmemCols = TN;
  static constexpr int kSmem = kStages * kStageBytes + 1024 /*alignment*/ + 256 /*barriers*/;
};

__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  return remote;
}
// TMA tile load of a CTA pair: the data lands in this CTA's shared memory, the bytes are counted on an
// mbarrier that may be the peer's (a shared::cluster address).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t holder, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T for one K step of 16 elements; issued by one thread of the leader.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}
// One arrival on the mbarrier at this shared-memory offset in both CTAs of the pair once all MMAs issued
// so far by this thread have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(both) : "memory");
}

template <int TN, int ST, typename Epi>
__global__ void __launch_bounds__(128) gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmW,
                                                       const __grid_constant__ CUtensorMap tmX /*box: TN/2 rows*/,
                                                       int M, int N, int nchunks, Epi epi, uint32_t* err) {
  using Cfg = GemmTc2Cfg<TN, ST>;
  constexpr int S = Cfg::kStages;
  constexpr uint32_t kWBytes = kGemmRowsW * kGemmBK * 2, kXBytes = Cfg::kXHalfBytes;
  constexpr int kRing = S * Cfg::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kRing;                    // full[S], empty[S], accum, tmem holder
  const uint32_t full0 = bars, empty0 = bars + 8 * S, accum_bar = bars + 16 * S, holder = bars + 16 * S + 8;
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(ring_ptr + kRing + 16 * S + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();                  // 0: leader
  const int n0 = blockIdx.x * kGemmRowsW, m0 = blockIdx.y * TN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(accum_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmX);
  }
  if (warp == 1) { tmem_alloc_pair(holder, Cfg::kTmemCols); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;

  if (warp == 0 && lane == 0) {
    // ---- TMA producer (both CTAs): own weight rows, own half of the token tile
    const int pre = nchunks < S ? nchunks : S;
    for (int i = 0; i < pre; ++i) {                      // weights do not depend on the upstream kernel
      if (rank == 0) mbar_expect_tx(full0 + 8 * i, 2 * (kWBytes + kXBytes));
      tma_load_3d_pair(base + i * Cfg::kStageBytes, &tmW, map_to_cta(full0 + 8 * i, 0), i * kGemmBK, n0, 0);
    }
    grid_dep_wait();
    for (int i = 0; i < pre; ++i)
      tma_load_3d_pair(base + i * Cfg::kStageBytes + kWBytes, &tmX, map_to_cta(full0 + 8 * i, 0), i * kGemmBK,
                       m0 + (int)rank * (TN / 2), 0);
    for (int i = pre; i < nchunks; ++i) {
      const int s = i % S;
      if (!mbar_wait(empty0 + 8 * s, ((i / S) - 1) & 1, err)) break;
      if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * (kWBytes + kXBytes));
      const uint32_t fb = map_to_cta(full0 + 8 * s, 0);
      tma_load_3d_pair(base + s * Cfg::kStageBytes, &tmW, fb, i * kGemmBK, n0, 0);
      tma_load_3d_pair(base + s * Cfg::kStageBytes + kWBytes, &tmX, fb, i * kGemmBK, m0 + (int)rank * (TN / 2), 0);
    }
  }
  if (warp == 1 && lane == 0 && rank == 0) {
    // ---- MMA issuer (leader only): 256 features x TN tokens per instruction
    constexpr uint32_t idesc = umma_idesc_bf16(2 * kGemmRowsW, TN);
    for (int i = 0; i < nchunks; ++i) {
      const int s = i % S;
      if (!mbar_wait(full0 + 8 * s, (i / S) & 1, err)) break;
      tc_fence_after();
      const uint32_t wa = base + s * Cfg::kStageBytes, xa = wa + kWBytes;
#pragma unroll
      for (int k = 0; k < kGemmBK / 16; ++k)
        umma_bf16_pair(tmem, umma_desc_k_sw128(wa + 32 * k), umma_desc_k_sw128(xa + 32 * k), idesc, (i | k) != 0);
      umma_commit_pair(empty0 + 8 * s);                  // the stage is reusable in both CTAs
    }
    umma_commit_pair(accum_bar);                         // both accumulators complete
  }
  __syncwarp();
  grid_dep_wait();
  const bool done = mbar_wait(accum_bar, 0, err);
  tc_fence_after();
  grid_dep_launch();

  // ---- epilogue: warp w reads TMEM lanes 32w .. 32w+31 (features n0 + 32w + lane) of this CTA
  const int n = n0 + 32 * warp + lane;
  const uint32_t trow = tmem + ((uint32_t)(32 * warp) << 16);
  if (done) {
#pragma unroll 1
    for (int c0 = 0; c0 < TN; c0 += 32) {
      float v[32];
      tmem_ld32(trow + c0, v);
      if (n < N && m0 + c0 < M) epi.template col<32>(0, m0 + c0, n, v, M - (m0 + c0));
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // neither CTA frees while the other still reads
  if (warp == 1) tmem_dealloc_pair(tmem, Cfg::kTmemCols);
}

}  // namespace vadusa

namespace vadusa {

// ---- persistent variant --------------------------------------------------------------------------
// The same CTA-pair product, but a pair stays resident and walks a list of output tiles (256 features x 256
// tokens each; tile t -> token tile t / (N / 256), feature pair t % (N / 256), so that the pairs running at the
// same time share token rows in L2): two accumulators of 256 columns in TMEM, so the epilogue of tile k (four
// warps of their own) runs under the main loop of tile k + 1, and the TMA ring (six stages of 32 KB) streams on
// across tile boundaries.  For products with at least two rounds of tiles per pair; one CTA per SM.
// Warps: 0 TMA producer (lane 0, both CTAs), 1 TMEM owner / MMA issuer (leader's lane 0), 2..9 epilogue (two warps
// per quarter of the TMEM lanes, half of the tile's tokens each: the epilogue, not the main loop, bounds a tile).
constexpr int kGemmP2Threads = 320;
constexpr int kGemmP2Stages = 6;
constexpr int kGemmP2TN = 256;
constexpr int kGemmP2StageBytes = kGemmRowsW * kGemmBK * 2 + (kGemmP2TN / 2) * kGemmBK * 2;      // 32 KB
constexpr int kGemmP2Smem = kGemmP2Stages * kGemmP2StageBytes + 1024 /*alignment*/ + 256 /*barriers*/;

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t remote_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}

template <typename Epi>
__global__ void __launch_bounds__(kGemmP2Threads, 1) gemm_tc2p_kernel(const __grid_constant__ CUtensorMap tmW,
                                                                      const __grid_constant__ CUtensorMap tmX /*box: 128 rows*/,
                                                                      int M, int N, int nchunks, int ntiles, Epi epi, uint32_t* err) {
  constexpr int S = kGemmP2Stages, TN = kGemmP2TN;
  constexpr uint32_t kWBytes = kGemmRowsW * kGemmBK * 2, kXBytes = (TN / 2) * kGemmBK * 2;
  constexpr int kRing = S * kGemmP2StageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kRing;        // full[S], empty[S], acc_full[2], acc_empty[2], tmem holder
  const uint32_t full0 = bars, empty0 = bars + 8 * S, accf0 = bars + 16 * S, acce0 = accf0 + 16, holder = acce0 + 16;
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(ring_ptr + kRing + 16 * S + 32);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();                  // 0: leader
  const int pair = (int)blockIdx.x >> 1, npairs = (int)gridDim.x >> 1;
  const int nfp = N / (2 * kGemmRowsW);                  // feature pairs per token tile
  const int my_tiles = pair < ntiles ? (ntiles - pair + npairs - 1) / npairs : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(accf0, 1); mbar_init(accf0 + 8, 1);
    mbar_init(acce0, 2); mbar_init(acce0 + 8, 2);        // one arrival per CTA of the pair
    mbar_fence_init();
    tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmX);
  }
  if (warp == 1) { tmem_alloc_pair(holder, 2 * TN); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer (both CTAs): own 128 weight rows, own half of the token tile; one chunk counter over all tiles
      bool waited = false, ok = true;
      long long g = 0;
      for (int k = 0; k < my_tiles && ok; ++k) {
        const int t = pair + k * npairs;
        const int n0 = (t % nfp) * 2 * kGemmRowsW + (int)rank * kGemmRowsW, m0 = (t / nfp) * TN + (int)rank * (TN / 2);
        for (int i = 0; i < nchunks; ++i, ++g) {
          const int s = (int)(g % S);
          if (g >= S && !mbar_wait(empty0 + 8 * s, (uint32_t)((g / S) - 1) & 1, err)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * (kWBytes + kXBytes));
          const uint32_t fb = map_to_cta(full0 + 8 * s, 0);
          tma_load_3d_pair(base + s * kGemmP2StageBytes, &tmW, fb, i * kGemmBK, n0, 0);
          if (!waited) { grid_dep_wait(); waited = true; }        // the tokens come from the upstream kernel
          tma_load_3d_pair(base + s * kGemmP2StageBytes + kWBytes, &tmX, fb, i * kGemmBK, m0, 0);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ---- MMA issuer (leader only): 256 features x 256 tokens per instruction, accumulator k & 1
      constexpr uint32_t idesc = umma_idesc_bf16(2 * kGemmRowsW, TN);
      bool ok = true;
      long long g = 0;
      for (int k = 0; k < my_tiles && ok; ++k) {
        const int b = k & 1;
        // both CTAs' epilogue warps have read what tile k - 2 left in this accumulator
        if (k >= 2 && !mbar_wait_cluster(acce0 + 8 * b, (uint32_t)((k >> 1) - 1) & 1, err)) break;
        tc_fence_after();
        for (int i = 0; i < nchunks; ++i, ++g) {
          const int s = (int)(g % S);
          if (!mbar_wait(full0 + 8 * s, (uint32_t)(g / S) & 1, err)) { ok = false; break; }
          tc_fence_after();
          const uint32_t wa = base + s * kGemmP2StageBytes, xa = wa + kWBytes;
#pragma unroll
          for (int kk = 0; kk < kGemmBK / 16; ++kk)
            umma_bf16_pair(tmem + TN * b, umma_desc_k_sw128(wa + 32 * kk), umma_desc_k_sw128(xa + 32 * kk), idesc, (i | kk) != 0);
          umma_commit_pair(empty0 + 8 * s);
        }
        if (ok) umma_commit_pair(accf0 + 8 * b);
      }
    }
  } else {
    // ---- epilogue warps: TMEM lanes 32 (warp % 4) .. +31 = features n0 + 32 (warp % 4) + lane of this CTA
    const int wq = warp & 3, chalf = (warp - 2) >> 2;
    grid_dep_wait();
    for (int k = 0; k < my_tiles; ++k) {
      const int t = pair + k * npairs, b = k & 1;
      const int n = (t % nfp) * 2 * kGemmRowsW + (int)rank * kGemmRowsW + 32 * wq + lane, m0 = (t / nfp) * TN;
      const bool done = mbar_wait(accf0 + 8 * b, (uint32_t)(k >> 1) & 1, err);
      tc_fence_after();
      if (k == my_tiles - 1) grid_dep_launch();
      const uint32_t trow = tmem + ((uint32_t)(32 * wq) << 16) + TN * b;
      if (done) {
#pragma unroll 1
        for (int c0 = chalf * (TN / 2); c0 < (chalf + 1) * (TN / 2); c0 += 32) {
          float v[32];
          tmem_ld32(trow + c0, v);
          if (n < N && m0 + c0 < M) epi.template col<32>(0, m0 + c0, n, v, M - (m0 + c0));
        }
      }
      // this CTA's eight epilogue warps are done with the accumulator: one arrival at the leader
      tc_fence_before();
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (threadIdx.x == 64) mbar_arrive_cluster(map_to_cta(acce0 + 8 * b, 0));
    }
    if (my_tiles == 0) grid_dep_launch();
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // neither CTA frees while the other still reads
  if (warp == 1) tmem_dealloc_pair(tmem, 2 * TN);
}

}  // namespace vadusa
