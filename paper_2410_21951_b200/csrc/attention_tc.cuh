// Tree-masked decode attention over the paged bf16 KV cache on the tcgen05 tensor cores
// (head_dim 64).  Node n of sequence b attends to every cached position < ctx_len[b] and to
// the tree slots ctx_len[b] + m whose bit m is set in anc[n] (paper Sec. II-A, tree attention).
//
// One CTA per (head, sequence, tile of 64 nodes, KV split); the splits of one (head, sequence, tile) form a
// cluster.  Trees of up to 128 nodes carry two 64-bit ancestor words per node.
// The 64 query rows are stored twice in the 128-row Q operand, so the scores of row r appear in
// TMEM lanes r and r + 64: warps 0-1 (lanes 0..63) work on keys 0..31 of every 64-key page,
// warps 2-3 (lanes 64..127) on keys 32..63.  Per page:
//   S = Q K^T      tcgen05.mma, A = Q tile, B = K tile, D in one of three TMEM score buffers (columns
//                  0..63 / 64..127 / 128..191), issued by a warp of its own up to three pages ahead of
//                  P V, so that neither the softmax nor the other issuer waits for it
//   softmax        each thread reads its 32 scores, keeps a scaling maximum of its own for its key
//                  half of the row, and the weights go back to TMEM as
//                  two bf16 halves (p = hi + lo, 16 significant bits) over the score columns,
//                  zero in the other thread's key range.  (Weights rounded to bf16 once would save the lo
//                  product, 4 % of a batch-64 launch, and take the logits of a 12-layer pass over contexts of
//                  up to 3000 tokens from 1.5e-2 to 2.05e-2 away from an fp64 evaluation.)
//   O += P V       tcgen05.mma with A from TMEM (hi then lo), B = V tile (MN-major), accumulating
//                  in TMEM columns 192..255; lanes r and r + 64 hold the two key-halves' sums
// The scaling maximum of a row only moves when the page maximum exceeds it by more than 2^6
// (p <= 64 is harmless in fp32 / bf16); then the row's accumulator is rescaled in TMEM.
// At the end rows r and r + 64 are brought to a common scale and added; splits are merged through an exchange area in global
// memory (L2) in a fixed order.
// K and V tiles have rings of their own: a K tile is free as soon as its Q K^T has completed, a V tile after
// its P V.  "Scores ready", "weights ready" and "P V done" have one mbarrier per score buffer: a buffer's next
// use cannot begin before the waiter of the current one has passed, so no parity wait can fall a round behind.
// Warps: 0-3 softmax, warp 4 lane 0 TMA producer, warp 5 TMEM owner / P V issuer, warp 6 Q K^T issuer.
#pragma once
#include "tc.cuh"

namespace vadusa {

constexpr int kAttStagesK = 4;                                               // K tiles leave their ring after Q K^T,
constexpr int kAttStagesV = 6;                                               // V tiles after P V: rings of their own
constexpr int kAttThreads = 224;
constexpr int kAttTileBytes = 64 * 64 * 2;                                   // one K or V page tile
constexpr int kAttRingBytes = (kAttStagesK + kAttStagesV) * kAttTileBytes;   // 80 KB; also holds the 64x64 fp32 output exchange
constexpr int kAttSmemBytes = 2 * kAttTileBytes /*Q, 128 rows*/ + kAttRingBytes + 1024 /*sums, maxima*/ +
                              1024 /*alignment*/ + 256 /*barriers*/;
constexpr float kAttRescaleStep = 6.0f;                                      // log2 units

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem] for one K step of 16 elements (A: lane = row, 8 columns of bf16 pairs).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two independent fp32 operations in one instruction (each half rounds as the scalar form does).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
__device__ __forceinline__ float2 fsub2(float2 a, float2 b) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "sub.rn.f32x2 rd, ra, rb;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kAttThreads) tree_attention_tc_kernel(
    const __grid_constant__ CUtensorMap tmQ,    // q [1][batch * n_nodes][d_model], box 64 x 64
    const __grid_constant__ CUtensorMap tmKV,   // pool [layers][blocks * 2 * heads * 64][64], box 64 x 64
    int layer, const int32_t* __restrict__ block_table, const int32_t* __restrict__ ctx_len,
    const int32_t* __restrict__ nvalid, const int32_t* __restrict__ order /*may be null*/, TreeView tree, KvGeom geom,
    int d_model, float scale_log2e, int splits,
    bf16* __restrict__ out, float* __restrict__ xch /*split exchange area*/, uint32_t* err) {
  constexpr int SK = kAttStagesK, SV = kAttStagesV;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_addr = base, ring = base + 2 * kAttTileBytes, ring_v = ring + SK * kAttTileBytes;
  uint8_t* ring_ptr = base_ptr + 2 * kAttTileBytes;
  float* lx = reinterpret_cast<float*>(ring_ptr + kAttRingBytes);            // end of the kernel: [128] partial sums, [128] scaling maxima
  const uint32_t bars = ring + kAttRingBytes + 1024;
  const uint32_t full_k0 = bars, empty_k0 = bars + 8 * SK, full_v0 = bars + 16 * SK, empty_v0 = full_v0 + 8 * SV,
                 bar_q = bars + 16 * (SK + SV), bar_s0 = bar_q + 8, bar_p0 = bar_q + 32,
                 bar_o0 = bar_q + 56, holder = bar_q + 80;     // scores ready / weights ready / P V done: one each per score
                                                               // buffer, so that a phase parity is never one round behind
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(ring_ptr + kAttRingBytes + 1024 + 16 * (SK + SV) + 80);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.x, split = blockIdx.z;
  const int N = tree.n_nodes;

  if (tid == 0) {
    for (int s = 0; s < 2 * (SK + SV); ++s) mbar_init(bars + 8 * s, 1);       // full / empty of the K and V rings
    mbar_init(bar_q, 1); mbar_init(bar_s0, 1); mbar_init(bar_s0 + 8, 1); mbar_init(bar_s0 + 16, 1);
    for (int j = 0; j < 3; ++j) { mbar_init(bar_p0 + 8 * j, 128); mbar_init(bar_o0 + 8 * j, 1); }
    mbar_fence_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmKV);
  }
  if (warp == 5) { tmem_alloc(holder, 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;

  grid_dep_wait();                            // q, K/V rows, lengths come from upstream kernels
  // blockIdx.y = (sequence, tile of 64 nodes); longest sequences first
  const int ntile = (N + 63) >> 6, qt = (int)blockIdx.y % ntile, node0 = 64 * qt;
  const int b = order ? order[blockIdx.y / ntile] : (int)blockIdx.y / ntile;
  const int nv = nvalid[b], ctx = ctx_len[b];
  const int total = ctx + nv;
  const int npages = nv > 0 ? (total + kKvBlock - 1) / kKvBlock : 0;
  const int per = (npages + splits - 1) / splits;
  const int p0 = split * per, p1 = min(npages, p0 + per);
  const int ntiles = max(0, p1 - p0);

  float m_use = -INFINITY, l_run = 0.f;       // softmax threads: scaling maximum (log2 units) and partial sum

  if (warp == 4) {
    // ---- TMA producer (lane 0); the block ids of this CTA's pages are fetched by the whole warp first
    long long blk_mine[2] = {0, 0};
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int i = lane + 32 * r;
      if (i < ntiles) {
        const long long v = kv_block_of(block_table, geom, b, (p0 + i) * kKvBlock, err);
        blk_mine[r] = v < 0 ? 0 : v;          // flagged; stay inside the pool
      }
    }
    if (lane == 0 && ntiles > 0) {
      mbar_expect_tx(bar_q, 2 * kAttTileBytes);
      tma_load_3d(q_addr, &tmQ, bar_q, h * 64, b * N + node0, 0);
      tma_load_3d(q_addr + kAttTileBytes, &tmQ, bar_q, h * 64, b * N + node0, 0);      // the same rows again: lanes 64..127
    }
    bool ok = true;
    for (int i = 0; i < ntiles; ++i) {
      long long blk;
      if (i < 64) {
        blk = __shfl_sync(0xffffffffu, (i < 32) ? blk_mine[0] : blk_mine[1], i & 31);
      } else {
        blk = kv_block_of(block_table, geom, b, (p0 + i) * kKvBlock, err);
        if (blk < 0) blk = 0;
      }
      if (lane == 0 && ok) {
        const int sk = i % SK, sv = i % SV;
        const int row = (int)((blk * 2 * geom.n_heads + h) * kKvBlock);
        if (i >= SK && !mbar_wait(empty_k0 + 8 * sk, ((i / SK) - 1) & 1, err)) {
          ok = false;                         // timed out (recorded): stop issuing, keep the warp converged
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
  } else if (warp == 5) {
    // ---- P V issuer (lane 0): O += P(i) V(i) as soon as the softmax threads have stored P(i)
    if (lane == 0) {
      constexpr uint32_t idesc_pv = umma_idesc_bf16(128, 64) | (1u << 16);     // B (V tile) is MN-major
      for (int i = 0; i < ntiles; ++i) {
        if (!mbar_wait(bar_p0 + 8 * (i % 3), (i / 3) & 1, err)) break;
        if (!mbar_wait(full_v0 + 8 * (i % SV), (i / SV) & 1, err)) break;
        tc_fence_after();
        const uint32_t va = ring_v + (i % SV) * kAttTileBytes, pa = tmem + 64 * (i % 3);
#pragma unroll
        for (int k = 0; k < 4; ++k)          // 16 keys per step: 8 TMEM columns of A, 16 rows (2048 bytes) of V
          umma_bf16_ts(tmem + 192, pa + 8 * k, umma_desc_k_sw128(va + 2048 * k), idesc_pv, (i | k) != 0);
#pragma unroll
        for (int k = 0; k < 4; ++k)          // the lo halves of the weights
          umma_bf16_ts(tmem + 192, pa + 32 + 8 * k, umma_desc_k_sw128(va + 2048 * k), idesc_pv, true);
        umma_commit(empty_v0 + 8 * (i % SV));
        umma_commit(bar_o0 + 8 * (i % 3));
      }
    }
  } else if (warp == 6) {
    // ---- Q K^T issuer (lane 0): S(i) = Q K(i)^T into score buffer i % 3, up to three pages ahead of P V
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 64);
      bool ok = ntiles == 0 || mbar_wait(bar_q, 0, err);
      for (int i = 0; i < ntiles && ok; ++i) {
        // the buffer held P(i - 3): free once P(i - 3) V(i - 3) has completed
        if (i >= 3 && !mbar_wait(bar_o0 + 8 * (i % 3), ((i - 3) / 3) & 1, err)) break;
        const int s = i % SK;
        if (!mbar_wait(full_k0 + 8 * s, (i / SK) & 1, err)) break;
        tc_fence_after();
        const uint32_t ka = ring + s * kAttTileBytes;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(tmem + 64 * (i % 3), umma_desc_k_sw128(q_addr + 32 * k), umma_desc_k_sw128(ka + 32 * k), idesc_qk, k != 0);
        umma_commit(empty_k0 + 8 * s);                     // the K tile is free once these MMAs have read it
        umma_commit(bar_s0 + 8 * (i % 3));
      }
    }
  } else {
    // ---- softmax: thread tid owns TMEM lane tid = query row (tid & 63), keys 32*half .. 32*half+31 of each page
    const int row = tid & 63, half = tid >> 6;
    unsigned long long alo = 0ull, ahi = 0ull;                     // ancestor-or-self bits of this row's node
    if (node0 + row < nv) tree.anc_of(b, node0 + row, alo, ahi);
    const uint32_t trow = tmem + ((uint32_t)(32 * warp) << 16);
    for (int i = 0; i < ntiles; ++i) {
      if (!mbar_wait(bar_s0 + 8 * (i % 3), (i / 3) & 1, err)) break;
      tc_fence_after();
      const uint32_t tsp = trow + 64 * (i % 3);       // this page's score / weight buffer
      float sc[32];
      tmem_ld32(tsp + 32 * half, sc);
      const int key0 = (p0 + i) * kKvBlock + 32 * half;
      if (key0 + 32 > ctx) {
        // bit j of vis: key key0 + j is visible (context, or an ancestor-or-self tree node; the ancestor
        // word has no bits at or above the node count).  Selects, not branches: the rows of a warp differ.
        const int rel = key0 - ctx;           // > -32 here
        uint32_t vis;
        if (rel >= 0) vis = rel < 128 ? bits32_at(alo, ahi, rel) : 0u;
        else vis = ((1u << (-rel)) - 1u) | (uint32_t)(alo << (-rel));
#pragma unroll
        for (int j = 0; j < 32; ++j) sc[j] = ((vis >> j) & 1u) ? sc[j] : -INFINITY;
      }                                       // else: all 32 keys inside the context, every key visible
      float mx4[4];                           // four chains of three-input maxima over eight scores each
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        mx4[c] = fmax3(sc[8 * c], sc[8 * c + 1], sc[8 * c + 2]);
        mx4[c] = fmax3(mx4[c], sc[8 * c + 3], sc[8 * c + 4]);
        mx4[c] = fmax3(mx4[c], sc[8 * c + 5], sc[8 * c + 6]);
        mx4[c] = fmaxf(mx4[c], sc[8 * c + 7]);
      }
      float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      if ((p0 + i + 1) * kKvBlock > total && tid < 64) {   // rows of V past the tree may hold anything: zero them
        const int valid = total - (p0 + i) * kKvBlock;
        mbar_wait(full_v0 + 8 * (i % SV), (i / SV) & 1, err);      // the V tile has landed before rows of it are cleared
        if (tid >= valid) {
          uint4* vr = reinterpret_cast<uint4*>(ring_ptr + (SK + i % SV) * kAttTileBytes + tid * 128);
#pragma unroll
          for (int c = 0; c < 8; ++c) vr[c] = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
      }
      // each key half of a row keeps its own scaling maximum (the halves accumulate in separate TMEM lanes
      // and are brought to a common scale once, at the end)
      mx *= scale_log2e;                      // raw scores; the (positive) scale moves into the exponent
      // move the scaling maximum only when the page maximum exceeds it by more than the step
      float factor = 1.f;
      if (mx > m_use + kAttRescaleStep || m_use == -INFINITY) {
        factor = (m_use == -INFINITY) ? 0.f : fast_exp2(m_use - mx);
        if (mx > -INFINITY) m_use = mx;
      }
      if (i > 0 && __any_sync(0xffffffffu, factor != 1.f)) {
        // rescale this row's accumulator, once the previous page's P V has completed
        if (!mbar_wait(bar_o0 + 8 * ((i - 1) % 3), ((i - 1) / 3) & 1, err)) break;
        tc_fence_after();
        float ot[32];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          tmem_ld32(trow + 192 + 32 * hh, ot);
          uint32_t ob[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) ob[e] = __float_as_uint(ot[e] * factor);
          tmem_st32(trow + 192 + 32 * hh, ob);
        }
      }
      l_run *= factor;
      float2 psum4[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};   // four chains of pairs
      uint32_t hv[16], lv[16];
      const float m_sub = (m_use == -INFINITY) ? 0.f : m_use;      // no visible key yet: every score is -inf, p = 0
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
      // this thread's 32 keys sit in columns 16*half .. 16*half+15 of each 32-column group; zero elsewhere
      {
        uint32_t zero[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) zero[j] = 0u;
        tmem_st16(tsp + 16 * half, hv);
        tmem_st16(tsp + 16 * (1 - half), zero);
        tmem_st16(tsp + 32 + 16 * half, lv);
        tmem_st16(tsp + 32 + 16 * (1 - half), zero);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bar_p0 + 8 * (i % 3));
    }
    if (ntiles > 0) { mbar_wait(bar_o0 + 8 * ((ntiles - 1) % 3), ((ntiles - 1) / 3) & 1, err); tc_fence_after(); }
  }
  __syncwarp();
  grid_dep_launch();
  __syncthreads();                            // the ring is idle from here on (every MMA has completed)

  // ---- output: rows r and r + 64 are the two key-halves of node r
  float* Ox = reinterpret_cast<float*>(ring_ptr);          // [64][64] fp32 exchange, row r rotated by 4r columns
  float o_acc[64];
  if (warp < 4) {
    const uint32_t trow = tmem + ((uint32_t)(32 * warp) << 16);
    if (ntiles > 0) {
      tmem_ld32(trow + 192, o_acc);
      tmem_ld32(trow + 224, o_acc + 32);
    } else {
#pragma unroll
      for (int e = 0; e < 64; ++e) o_acc[e] = 0.f;
    }
    lx[tid] = l_run;
    lx[128 + tid] = m_use;
    if (tid >= 64) {
#pragma unroll
      for (int e = 0; e < 64; ++e) Ox[(tid - 64) * 64 + ((e + 4 * tid) & 63)] = o_acc[e];
    }
  }
  __syncthreads();
  if (tid < 64) {
    // the two key halves of the row on a common scale
    const float m1 = lx[128 + tid + 64], mm = fmaxf(m_use, m1);
    const float w0 = (m_use == -INFINITY) ? 0.f : fast_exp2(m_use - mm), w1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - mm);
#pragma unroll
    for (int e = 0; e < 64; ++e) o_acc[e] = o_acc[e] * w0 + Ox[tid * 64 + ((e + 4 * tid) & 63)] * w1;
    l_run = l_run * w0 + lx[tid + 64] * w1;
    m_use = mm;
  }
  if (splits == 1) {
    if (tid < 64 && node0 + tid < N) {
      const float inv = (node0 + tid < nv && l_run > 0.f) ? 1.f / l_run : 0.f;
      uint4* dst = reinterpret_cast<uint4*>(out + ((long long)b * N + node0 + tid) * d_model + h * 64);
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
  } else {
    // this split's result goes to its slot of the exchange area in global memory (it stays in L2):
    // O [64 nodes][64] fp32, then the row sums l[64] and scaling maxima m[64]; the splits of one (head,
    // sequence) meet at a cluster barrier and are merged in a fixed order
    constexpr int kSlot = 64 * 64 + 128;
    float* mine = xch + ((long long)(blockIdx.y * gridDim.x + blockIdx.x) * splits + split) * kSlot;
    if (tid < 64) {
      float4* dst = reinterpret_cast<float4*>(mine + tid * 64);
#pragma unroll
      for (int c = 0; c < 16; ++c) dst[c] = make_float4(o_acc[4 * c], o_acc[4 * c + 1], o_acc[4 * c + 2], o_acc[4 * c + 3]);
      mine[64 * 64 + tid] = l_run;
      mine[64 * 64 + 64 + tid] = m_use;
    }
    cluster_sync_all();                        // release / acquire: the peers' slots are visible
    // CTA `split` finishes nodes [split*per_n, (split+1)*per_n): 16 threads per node, four consecutive
    // features each
    const float* first = xch + (long long)(blockIdx.y * gridDim.x + blockIdx.x) * splits * kSlot;
    const int per_n = 64 / splits;
    if (tid < 128) {
      const int e4 = (tid & 15) * 4;
      for (int n = split * per_n + (tid >> 4); n < (split + 1) * per_n; n += 8) {
        float mm[8], ll[8];
        float4 oo[8];
        float M = -INFINITY;
#pragma unroll
        for (int p = 0; p < 8; ++p)
          if (p < splits) {
            const float* sl = first + (long long)p * kSlot;
            mm[p] = __ldcg(sl + 64 * 64 + 64 + n);
            ll[p] = __ldcg(sl + 64 * 64 + n);
            oo[p] = __ldcg(reinterpret_cast<const float4*>(sl + n * 64 + e4));
            M = fmaxf(M, mm[p]);
          }
        float L = 0.f;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int p = 0; p < 8; ++p)
          if (p < splits) {
            const float w = (mm[p] == -INFINITY) ? 0.f : exp2f(mm[p] - M);
            L = fmaf(ll[p], w, L);
            o.x = fmaf(oo[p].x, w, o.x); o.y = fmaf(oo[p].y, w, o.y); o.z = fmaf(oo[p].z, w, o.z); o.w = fmaf(oo[p].w, w, o.w);
          }
        if (node0 + n < N) {
          const float inv = (node0 + n < nv && L > 0.f) ? 1.f / L : 0.f;
          uint2 v;
          v.x = pack_bf16(o.x * inv, o.y * inv);
          v.y = pack_bf16(o.z * inv, o.w * inv);
          *reinterpret_cast<uint2*>(out + ((long long)b * N + node0 + n) * d_model + h * 64 + e4) = v;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 256);
}

}  // namespace vadusa
