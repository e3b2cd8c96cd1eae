// Causal attention of prefix chunks over the paged bf16 KV cache on the tcgen05 tensor cores (head_dim 64):
// the prefilling pass over [phonemes ; prompt] (paper Fig. 1a, Sec. II-A), whose rows are chunks of 64
// consecutive tokens of a sequence.  Two consecutive chunks of one sequence share a CTA: 128 distinct query
// rows (the MMA's full height) against every K/V page, so each page is fetched once per 128 queries instead
// of once per 64, and the weights of a row fill a whole TMEM lane (no duplicated rows, no zero halves).
//
// Row r of chunk c sits at absolute position ctx_len[c] + r and sees every key at a position <= its own
// (the chunk's K/V rows are in the cache before the pass's attention starts).  The second chunk of a pair
// starts 64 positions behind the first (the host pairs only such chunks); a pair may lack its second chunk.
// Per 64-key page:  S = Q K^T (128 x 64) -> two threads per row (eight softmax warps): each reads all 64
// scores of the row for the scaling maximum (so both use the same one without talking to each other; it moves
// lazily, as in the tree kernel), masks by position, exponentiates its own 32 keys and writes the weights as two
// bf16 halves (hi, lo) over the scores once all softmax threads have read them (a named barrier per page)
// -> O += P V.  TMEM: three score / weight buffers (columns 0..191), O (192..255): two CTAs per SM.  Rings, barriers and bounded waits are those of tree_attention_tc_kernel.
// Warps: 0-7 softmax (warp w and w + 4 share TMEM lanes 32 (w % 4) ..), 8 TMA producer, 9 TMEM owner / P V issuer,
// 10 Q K^T issuer.
#pragma once
#include "attention_tc.cuh"

namespace vadusa {

constexpr int kPfThreads = 352;

// Two 32-column loads (32 lanes x 32 fp32 each) issued back to back, one wait for both.
__device__ __forceinline__ void tmem_ld32x2(uint32_t ta, float* a, uint32_t tb, float* b) {
  uint32_t r[32], q[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(ta)
      : "memory");
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(q[0]), "=r"(q[1]), "=r"(q[2]), "=r"(q[3]), "=r"(q[4]), "=r"(q[5]), "=r"(q[6]), "=r"(q[7]),
        "=r"(q[8]), "=r"(q[9]), "=r"(q[10]), "=r"(q[11]), "=r"(q[12]), "=r"(q[13]), "=r"(q[14]), "=r"(q[15]),
        "=r"(q[16]), "=r"(q[17]), "=r"(q[18]), "=r"(q[19]), "=r"(q[20]), "=r"(q[21]), "=r"(q[22]), "=r"(q[23]),
        "=r"(q[24]), "=r"(q[25]), "=r"(q[26]), "=r"(q[27]), "=r"(q[28]), "=r"(q[29]), "=r"(q[30]), "=r"(q[31])
      : "r"(tb)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) { a[i] = __uint_as_float(r[i]); b[i] = __uint_as_float(q[i]); }
}

__global__ void __launch_bounds__(kPfThreads, 2) prefill_attention_tc_kernel(
    const __grid_constant__ CUtensorMap tmQ,    // q [1][rows * 64][d_model], box 64 x 64
    const __grid_constant__ CUtensorMap tmKV,   // pool [layers][blocks * 2 * heads * 64][64], box 64 x 64
    int layer, const int32_t* __restrict__ block_table /*[rows][max_blocks]*/, const int32_t* __restrict__ ctx_len,
    const int32_t* __restrict__ nvalid, const int2* __restrict__ pairs /*[gridDim.y]: the tile's two rows (y < 0: none)*/,
    KvGeom geom, int d_model, float scale_log2e, bf16* __restrict__ out, uint32_t* err) {
  constexpr int SK = kAttStagesK, SV = kAttStagesV;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_addr = base, ring = base + 2 * kAttTileBytes, ring_v = ring + SK * kAttTileBytes;
  uint8_t* ring_ptr = base_ptr + 2 * kAttTileBytes;
  const uint32_t bars = ring + kAttRingBytes + 1024;
  const uint32_t full_k0 = bars, empty_k0 = bars + 8 * SK, full_v0 = bars + 16 * SK, empty_v0 = full_v0 + 8 * SV,
                 bar_q = bars + 16 * (SK + SV), bar_s0 = bar_q + 8, bar_p0 = bar_q + 32, bar_o0 = bar_q + 56, holder = bar_q + 80;
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(ring_ptr + kAttRingBytes + 1024 + 16 * (SK + SV) + 80);
  volatile int* s_abort = reinterpret_cast<volatile int*>(ring_ptr + kAttRingBytes + 1024 + 16 * (SK + SV) + 84);   // a wait of the softmax threads ran out

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.x;

  if (tid == 0) {
    for (int s = 0; s < 2 * (SK + SV); ++s) mbar_init(bars + 8 * s, 1);
    mbar_init(bar_q, 1); mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1); mbar_init(bar_s0 + 16, 1);
    for (int j = 0; j < 3; ++j) { mbar_init(bar_p0 + 8 * j, 256); mbar_init(bar_o0 + 8 * j, 1); }
    *s_abort = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmKV);
  }
  if (warp == 9) { tmem_alloc(holder, 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;

  grid_dep_wait();                            // q, K/V rows, lengths come from upstream kernels
  const int2 pr = pairs[blockIdx.y];
  const int rA = pr.x, rB = pr.y;
  const int ctxA = ctx_len[rA], nvA = nvalid[rA];
  const int ctxB = rB >= 0 ? ctx_len[rB] : 0, nvB = rB >= 0 ? nvalid[rB] : 0;
  const int total = max(nvA > 0 ? ctxA + nvA : 0, nvB > 0 ? ctxB + nvB : 0);
  const int ntiles = (total + kKvBlock - 1) / kKvBlock;

  float m_use = -INFINITY, l_run = 0.f;       // softmax threads: scaling maximum (log2 units) and sum of weights

  if (warp == 8) {
    // ---- TMA producer (lane 0)
    long long blk_mine[2] = {0, 0};
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int i = lane + 32 * r;
      if (i < ntiles) {
        const long long v = kv_block_of(block_table, geom, rA, i * kKvBlock, err);
        blk_mine[r] = v < 0 ? 0 : v;
      }
    }
    if (lane == 0 && ntiles > 0) {
      mbar_expect_tx(bar_q, 2 * kAttTileBytes);
      tma_load_3d(q_addr, &tmQ, bar_q, h * 64, rA * 64, 0);
      tma_load_3d(q_addr + kAttTileBytes, &tmQ, bar_q, h * 64, (rB >= 0 ? rB : rA) * 64, 0);
    }
    bool ok = true;
    for (int i = 0; i < ntiles; ++i) {
      long long blk;
      if (i < 64) {
        blk = __shfl_sync(0xffffffffu, (i < 32) ? blk_mine[0] : blk_mine[1], i & 31);
      } else {
        blk = kv_block_of(block_table, geom, rA, i * kKvBlock, err);
        if (blk < 0) blk = 0;
      }
      if (lane == 0 && ok) {
        const int sk = i % SK, sv = i % SV;
        const int row = (int)((blk * 2 * geom.n_heads + h) * kKvBlock);
        if (i >= SK && !mbar_wait(empty_k0 + 8 * sk, ((i / SK) - 1) & 1, err)) {
          ok = false;
        } else {
          mbar_expect_tx(full_k0 + 8 * sk, kAttTileBytes);
          tma_load_3d(ring + sk * kAttTileBytes, &tmKV, full_k0 + 8 * sk, 0, row, layer);
        }
        if (ok && i >= SV && !mbar_wait(empty_v0 + 8 * sv, ((i / SV) - 1) & 1, err)) ok = false;
        if (ok) {
          mbar_expect_tx(full_v0 + 8 * sv, kAttTileBytes);
          tma_load_3d(ring_v + sv * kAttTileBytes, &tmKV, full_v0 + 8 * sv, 0, row + geom.n_heads * kKvBlock, layer);
        }
      }
    }
  } else if (warp == 9) {
    // ---- P V issuer (lane 0)
    if (lane == 0) {
      constexpr uint32_t idesc_pv = umma_idesc_bf16(128, 64) | (1u << 16);     // B (V tile) is MN-major
      for (int i = 0; i < ntiles; ++i) {
        if (!mbar_wait(bar_p0 + 8 * (i % 3), (i / 3) & 1, err)) break;
        if (!mbar_wait(full_v0 + 8 * (i % SV), (i / SV) & 1, err)) break;
        tc_fence_after();
        const uint32_t va = ring_v + (i % SV) * kAttTileBytes, pa = tmem + 64 * (i % 3);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16_ts(tmem + 192, pa + 8 * k, umma_desc_k_sw128(va + 2048 * k), idesc_pv, (i | k) != 0);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16_ts(tmem + 192, pa + 32 + 8 * k, umma_desc_k_sw128(va + 2048 * k), idesc_pv, true);
        umma_commit(empty_v0 + 8 * (i % SV));
        umma_commit(bar_o0 + 8 * (i % 3));
      }
    }
  } else if (warp == 10) {
    // ---- Q K^T issuer (lane 0)
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 64);
      bool ok = ntiles == 0 || mbar_wait(bar_q, 0, err);
      for (int i = 0; i < ntiles && ok; ++i) {
        // score buffer i % 3 held the weights of page i - 3: free once that page's P V has completed
        if (i >= 3 && !mbar_wait(bar_o0 + 8 * (i % 3), ((i - 3) / 3) & 1, err)) break;
        const int s = i % SK;
        if (!mbar_wait(full_k0 + 8 * s, (i / SK) & 1, err)) break;
        tc_fence_after();
        const uint32_t ka = ring + s * kAttTileBytes;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(tmem + 64 * (i % 3), umma_desc_k_sw128(q_addr + 32 * k), umma_desc_k_sw128(ka + 32 * k), idesc_qk, k != 0);
        umma_commit(empty_k0 + 8 * s);
        umma_commit(bar_s0 + 8 * (i % 3));
      }
    }
  } else {
    // ---- softmax: threads (warp w, lane) and (warp w + 4, lane) own TMEM lane 32 (w % 4) + lane = row r of chunk
    // (lane >> 6); the first takes keys 0..31 of every page, the second keys 32..63
    const int tl = 32 * (warp & 3) + lane, khalf = warp >> 2;
    const int r = tl & 63, second = tl >> 6;
    const int nv_h = second ? nvB : nvA;
    const int qpos = (second ? ctxB : ctxA) + r;                  // this row's own position: the last key it sees
    const bool live = r < nv_h;
    const uint32_t trow = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
    // The softmax threads meet at a named barrier on every page, so none of them may leave the loop early: after a
    // wait has run out (recorded in the error word) the remaining waits return at once and the loop runs to its end.
    auto wait_ok = [&](uint32_t bar, uint32_t parity) -> bool {
      if (*s_abort) return false;
      if (mbar_wait(bar, parity, err)) return true;
      *s_abort = 1;
      return false;
    };
    for (int i = 0; i < ntiles; ++i) {
      wait_ok(bar_s0 + 8 * (i % 3), (i / 3) & 1);
      tc_fence_after();
      const uint32_t tsp = trow + 64 * (i % 3), tpp = tsp;       // the weights go over the scores
      // keys i*64 + j with j < nvis are visible
      const int nvis = live ? min(max(qpos - i * kKvBlock + 1, 0), kKvBlock) : 0;
      float sc[32], mx;
      {
        float so[32];                                             // the other thread's keys: for the maximum only
        tmem_ld32x2(tsp + 32 * khalf, sc, tsp + 32 * (1 - khalf), so);
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (nvis < kKvBlock) {                                    // (a page on or past the row's diagonal)
          const int no = nvis - 32 * (1 - khalf), nm = nvis - 32 * khalf;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            sc[j] = j < nm ? sc[j] : -INFINITY;
            so[j] = j < no ? so[j] : -INFINITY;
          }
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) mx4[j & 3] = fmax3(mx4[j & 3], sc[j], so[j]);
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      }
      // every softmax thread has the scores in registers: the buffer may now take the weights
      asm volatile("bar.sync 2, 256;" ::: "memory");
      if ((i + 1) * kKvBlock > total && tid < 64) {      // rows of V past the last token may hold anything: zero them
        const int valid = total - i * kKvBlock;
        wait_ok(full_v0 + 8 * (i % SV), (i / SV) & 1);
        if (tid >= valid) {
          uint4* vr = reinterpret_cast<uint4*>(ring_ptr + (SK + i % SV) * kAttTileBytes + tid * 128);
#pragma unroll
          for (int c = 0; c < 8; ++c) vr[c] = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
      }
      mx *= scale_log2e;
      float factor = 1.f;
      if (mx > m_use + kAttRescaleStep || m_use == -INFINITY) {
        factor = (m_use == -INFINITY) ? 0.f : fast_exp2(m_use - mx);
        if (mx > -INFINITY) m_use = mx;
      }
      if (i > 0 && __any_sync(0xffffffffu, factor != 1.f)) {
        // (both threads of a row see the same maxima, so they take this branch together: each rescales half of O)
        wait_ok(bar_o0 + 8 * ((i - 1) % 3), ((i - 1) / 3) & 1);
        tc_fence_after();
        float ot[32];
        tmem_ld32(trow + 192 + 32 * khalf, ot);
        uint32_t ob[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) ob[e] = __float_as_uint(ot[e] * factor);
        tmem_st32(trow + 192 + 32 * khalf, ob);
      }
      l_run *= factor;
      const float m_sub = (m_use == -INFINITY) ? 0.f : m_use;
      float2 psum4[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};   // four chains of pairs
      uint32_t hv[16], lv[16];
      const float2 sc2 = make_float2(scale_log2e, scale_log2e), nm2 = make_float2(-m_sub, -m_sub);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        // two keys per instruction where the pipe has a paired form (fma, add, sub)
        const float2 x = ffma2(make_float2(sc[2 * j], sc[2 * j + 1]), sc2, nm2);
        const float2 pp = make_float2(fast_exp2(x.x), fast_exp2(x.y));
        psum4[j & 3] = fadd2(psum4[j & 3], pp);
        hv[j] = pack_bf16(pp.x, pp.y);
        const float2 hh = make_float2(__uint_as_float(hv[j] << 16), __uint_as_float(hv[j] & 0xffff0000u));
        const float2 ll = fsub2(pp, hh);
        lv[j] = pack_bf16(ll.x, ll.y);
      }
      {
        const float2 s01 = fadd2(psum4[0], psum4[1]), s23 = fadd2(psum4[2], psum4[3]);
        const float2 st = fadd2(s01, s23);
        l_run += st.x + st.y;
      }
      tmem_st16(tpp + 16 * khalf, hv);                   // keys 32 khalf .. +31: hi in columns 16 khalf .., lo in 32 + 16 khalf ..
      tmem_st16(tpp + 32 + 16 * khalf, lv);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bar_p0 + 8 * (i % 3));
    }
    if (ntiles > 0) { wait_ok(bar_o0 + 8 * ((ntiles - 1) % 3), ((ntiles - 1) / 3) & 1); tc_fence_after(); }
  }
  __syncwarp();
  grid_dep_launch();
  __syncthreads();

  // ---- output: the two threads of a row add their sums of weights; the first writes the row
  float* lx = reinterpret_cast<float*>(ring_ptr);            // [128] (the ring is idle: every MMA has completed)
  if (warp >= 4 && warp < 8) lx[32 * (warp & 3) + lane] = l_run;
  __syncthreads();
  if (warp < 4) {
    const int tl = 32 * warp + lane, r = tl & 63, second = tl >> 6;
    const int row = second ? rB : rA, nv_h = second ? nvB : nvA;
    if (row >= 0) {
      const uint32_t trow = tmem + ((uint32_t)(32 * warp) << 16);
      float o_acc[64];
      if (ntiles > 0) {
        tmem_ld32(trow + 192, o_acc);
        tmem_ld32(trow + 224, o_acc + 32);
      } else {
#pragma unroll
        for (int e = 0; e < 64; ++e) o_acc[e] = 0.f;
      }
      const float l_all = l_run + lx[tl];
      const float inv = (r < nv_h && l_all > 0.f) ? 1.f / l_all : 0.f;
      uint4* dst = reinterpret_cast<uint4*>(out + ((long long)row * 64 + r) * d_model + h * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint4 v;
        v.x = pack_bf16(o_acc[8 * c + 0] * inv, o_acc[8 * c + 1] * inv);
        v.y = pack_bf16(o_acc[8 * c + 2] * inv, o_acc[8 * c + 3] * inv);
        v.z = pack_bf16(o_acc[8 * c + 4] * inv, o_acc[8 * c + 5] * inv);
        v.w = pack_bf16(o_acc[8 * c + 6] * inv, o_acc[8 * c + 7] * inv);
        dst[c] = v;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, 256);
}

}  // namespace vadusa
