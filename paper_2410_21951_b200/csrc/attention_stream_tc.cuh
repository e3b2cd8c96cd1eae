// Tree-masked decode attention for batches: one persistent kernel over the whole stream of K/V pages.
// (Paper Sec. II-A, tree attention; the same arithmetic as tree_attention_tc_kernel, page by page.)
//
// The pages of all sequences of the batch, sequence after sequence, form one stream of P pages.  The grid is
// made of groups of H CTAs (H heads); group j of G takes the pages [j P / G, (j + 1) P / G) and its CTA h works
// on head h of them: every CTA streams the same number of pages whatever the lengths of the sequences, the K/V
// rings never drain between sequences, tensor memory, the barriers and the launch are paid once, and the H CTAs
// of a group, walking the same pages at the same pace, ask DRAM for runs of H adjacent tiles (a page's K tiles
// of all heads are contiguous, and so are its V tiles).  A group's range is cut into segments, one per sequence
// it touches.  A segment that covers its whole sequence writes the (sequence, head) output; otherwise the
// segment leaves (O, l, m) in an exchange slot, and the part that arrives last (a counter per (sequence, head),
// no waiting) merges all parts in a fixed order and writes the output.
//
// Per page the work is that of tree_attention_tc_kernel: S = Q K^T into one of three TMEM score buffers,
// softmax by 128 threads (lanes r and r + 64 are the two key halves of query row r), weights back to TMEM as
// bf16 hi + lo, O += P V with A from TMEM.  (Weights rounded to bf16 once save a third of a page's tensor-core
// instructions and 15 % of a launch, but take the logits of a 12-layer pass over contexts of up to 3000 tokens
// from 1.5e-2 to 2.05e-2 away from an fp64 evaluation.)  The Q tile has two buffers: the next item's Q arrives while the
// current item runs, and the buffer of the finished item carries the exchange of the two key halves.
// Warps: 0-3 softmax and epilogue, warp 4 TMA producer of Q and K, warp 5 TMEM owner / P V issuer, warp 6 Q K^T
// issuer, warp 7 TMA producer of V.
// After a timeout the softmax warps run their loops to the end (they meet at named barriers).
#pragma once
#include "attention_tc.cuh"

namespace vadusa {

constexpr int kAsStagesK = 4, kAsStagesV = 5;
constexpr int kAsMaxBatch = 512;
constexpr int kAsThreads = 256;
constexpr int kAsGrid = 296;                                                  // two CTAs on each of 148 SMs
constexpr int kAsRingBytes = (kAsStagesK + kAsStagesV) * kAttTileBytes;
constexpr int kAsQBytes = 2 * kAttTileBytes;                                  // one Q buffer: the 64 rows twice
constexpr int kAsSmemBytes = 2 * kAsQBytes + kAsRingBytes + 1024 /*sums, maxima*/ + 2 * (kAsMaxBatch + 1) * 4 +
                             1024 /*alignment*/ + 384 /*barriers*/;
constexpr int kAsSlotFloats = 64 * 64 + 128;                                   // O, l, m of one part

// One segment: pages [p0, p1) of sequence b, which has np pages and is cut into `parts` parts, the first of them
// in group `first_grp`.
struct StreamSeg {
  int b, p0, p1, np, parts, part, first_grp;
  bool first_of_cta, part0_first;             // part0_first: part 0 is the first segment of its CTA (else the last)
};

// Walks the segments of one group's range of the stream of sequence pages.  cum[b] = pages of the sequences
// before b (in shared memory).  Group c of G takes the pages [c P / G, (c + 1) P / G).
struct StreamIter {
  const int* cum;
  int G, c, b;
  long long P, cur, lo, hi;
  bool first;
  __device__ void init(const int* cum_, int batch, int G_, int c_) {
    cum = cum_; G = G_; c = c_;
    P = cum[batch];
    first = true; b = 0;
    if (P < G) G = (int)P;                     // fewer pages than groups: one page each for the first P, so that no
    if (c >= G) { lo = hi = cur = 0; return; } // group between two parts of a sequence is empty
    lo = (long long)c * P / G;
    hi = (long long)(c + 1) * P / G;
    cur = lo;
    int a = 0, z = batch;                      // largest b with cum[b] <= lo
    while (z - a > 1) {
      const int m = (a + z) >> 1;
      if (cum[m] <= lo) a = m; else z = m;
    }
    b = a;
  }
  __device__ long long grp_lo(int grp) const { return (long long)grp * P / G; }
  __device__ bool next(StreamSeg& s) {
    if (cur >= hi) return false;
    while (cum[b + 1] <= cur) ++b;            // also steps over sequences without pages
    const long long S = cum[b], E = cum[b + 1];
    const long long end = hi < E ? hi : E;
    s.b = b; s.np = (int)(E - S);
    s.p0 = (int)(cur - S); s.p1 = (int)(end - S);
    const int cf = (int)(((S + 1) * G - 1) / P), cl = (int)((E * G - 1) / P);      // groups of the first and last page
    s.parts = cl - cf + 1; s.part = c - cf; s.first_grp = cf;
    s.part0_first = grp_lo(cf) == S;
    s.first_of_cta = first;
    first = false;
    cur = end;
    return true;
  }
};

__device__ __forceinline__ void as_bar128(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

__global__ void __launch_bounds__(kAsThreads, 2) tree_attention_stream_kernel(
    const __grid_constant__ CUtensorMap tmQ,    // q [1][batch * n_nodes][d_model], box 64 x 64
    const __grid_constant__ CUtensorMap tmKV,   // pool [layers][blocks * 2 * heads * 64][64], box 64 x 64
    int layer, const int32_t* __restrict__ block_table, const int32_t* __restrict__ ctx_len,
    const int32_t* __restrict__ nvalid, TreeView tree, KvGeom geom, int batch, int d_model, float scale_log2e,
    bf16* __restrict__ out, float* __restrict__ xch /*2 gridDim.x slots*/, uint32_t* __restrict__ cnt /*2 gridDim.x, zero*/,
    uint32_t* err) {
  constexpr int SK = kAsStagesK, SV = kAsStagesV;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_addr = base, ring = base + 2 * kAsQBytes, ring_v = ring + SK * kAttTileBytes;
  uint8_t* ring_ptr = base_ptr + 2 * kAsQBytes;
  float* lx = reinterpret_cast<float*>(ring_ptr + kAsRingBytes);             // [128] partial sums, [128] scaling maxima
  int* cum = reinterpret_cast<int*>(ring_ptr + kAsRingBytes + 1024);         // [batch + 1] pages before each sequence
  uint32_t* meta = reinterpret_cast<uint32_t*>(cum + kAsMaxBatch + 1);       // [batch] context length | nodes << 24
  constexpr int kBarOff = kAsRingBytes + 1024 + 2 * (kAsMaxBatch + 1) * 4;
  const uint32_t bars = ring + kBarOff;
  const uint32_t full_k0 = bars, empty_k0 = bars + 8 * SK, full_v0 = bars + 16 * SK, empty_v0 = full_v0 + 8 * SV,
                 q_full0 = bars + 16 * (SK + SV), q_empty0 = q_full0 + 16, bar_s0 = q_full0 + 32, bar_p0 = q_full0 + 56,
                 bar_o0 = q_full0 + 80, holder = q_full0 + 104;
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(ring_ptr + kBarOff + 16 * (SK + SV) + 104);
  volatile int* s_abort = reinterpret_cast<volatile int*>(holder_ptr + 1);   // a softmax wait ran out
  volatile int* s_flag = reinterpret_cast<volatile int*>(holder_ptr + 2);    // this CTA merges the item's parts

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = tree.n_nodes, H = geom.n_heads;
  // CTA c works on head c % H for group c / H: the H CTAs of a group walk the same pages of the same sequences at
  // the same time, so that what is in flight in DRAM at any moment are runs of H adjacent K (and V) tiles
  const int c = blockIdx.x, h = c % H, grp = c / H, ngroups = (int)gridDim.x / H;

  if (tid == 0) {
    for (int s = 0; s < 2 * (SK + SV); ++s) mbar_init(bars + 8 * s, 1);       // full / empty of the K and V rings
    for (int j = 0; j < 2; ++j) { mbar_init(q_full0 + 8 * j, 1); mbar_init(q_empty0 + 8 * j, 1); }
    for (int j = 0; j < 3; ++j) { mbar_init(bar_s0 + 8 * j, 1); mbar_init(bar_p0 + 8 * j, 128); mbar_init(bar_o0 + 8 * j, 1); }
    *s_abort = 0;
    *s_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmKV);
  }
  if (warp == 5) { tmem_alloc(holder, 256); tmem_relinquish(); }

  grid_dep_wait();                            // q, K/V rows, lengths come from upstream kernels
  for (int b = tid; b < batch; b += kAsThreads) {
    const int nv = nvalid[b], cx = ctx_len[b];
    meta[b] = (uint32_t)cx | ((uint32_t)nv << 24);
    cum[b + 1] = nv > 0 ? (cx + nv + kKvBlock - 1) / kKvBlock : 0;
  }
  if (tid == 0) cum[0] = 0;
  __syncthreads();
  if (warp == 0) {                            // running sum of the page counts
    int carry = 0;
    for (int b0 = 0; b0 < batch; b0 += 32) {
      int v = b0 + lane < batch ? cum[1 + b0 + lane] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
      }
      v += carry;
      if (b0 + lane < batch) cum[1 + b0 + lane] = v;
      carry = __shfl_sync(0xffffffffu, v, 31);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;

  StreamIter it;
  it.init(cum, batch, ngroups, grp);
  StreamSeg sg;

  if (warp == 4 || warp == 7) {
    // ---- TMA producers (lane 0 of each): warp 4 loads Q and the K tiles, warp 7 the V tiles, so that neither ring
    // waits for the other's slot; the block ids of a segment's pages are fetched by the whole warp first
    const bool is_k = warp == 4;
    const int stages = is_k ? SK : SV;
    const uint32_t full0 = is_k ? full_k0 : full_v0, empty0 = is_k ? empty_k0 : empty_v0, ring0 = is_k ? ring : ring_v;
    const int row_add = (is_k ? h : geom.n_heads + h) * kKvBlock;
    bool ok = true;
    int st = 0, s = 0;                         // ring stage of the next page, segments so far
    uint32_t ph = 1;                           // parity to wait for on the stage's "empty" barrier: passes at once in
    while (it.next(sg)) {                      // the ring's first round (no phase of it has completed yet)
      const int ntiles = sg.p1 - sg.p0;
      int row_mine[2] = {0, 0};
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int i = lane + 32 * r;
        if (i < ntiles) {
          const long long v = kv_block_of(block_table, geom, sg.b, (sg.p0 + i) * kKvBlock, err);
          row_mine[r] = (int)(v < 0 ? 0 : v) * 2 * geom.n_heads * kKvBlock + row_add;   // flagged; stay inside the pool
        }
      }
      if (is_k && lane == 0 && ok) {
        // the buffer held Q of the segment before the previous one: free once that segment's epilogue is over
        if (s >= 2 && !mbar_wait(q_empty0 + 8 * (s & 1), ((s >> 1) - 1) & 1, err)) ok = false;
        if (ok) {
          const uint32_t qa = q_addr + (s & 1) * kAsQBytes;
          mbar_expect_tx(q_full0 + 8 * (s & 1), kAsQBytes);
          tma_load_3d(qa, &tmQ, q_full0 + 8 * (s & 1), h * 64, sg.b * N, 0);
          tma_load_3d(qa + kAttTileBytes, &tmQ, q_full0 + 8 * (s & 1), h * 64, sg.b * N, 0);   // the same rows again: lanes 64..127
        }
      }
      for (int i = 0; i < ntiles; ++i) {
        int row;
        if (i < 64) {
          row = __shfl_sync(0xffffffffu, (i < 32) ? row_mine[0] : row_mine[1], i & 31);
        } else {
          const long long v = kv_block_of(block_table, geom, sg.b, (sg.p0 + i) * kKvBlock, err);
          row = (int)(v < 0 ? 0 : v) * 2 * geom.n_heads * kKvBlock + row_add;
        }
        if (lane == 0 && ok) {
          if (!mbar_wait(empty0 + 8 * st, ph, err)) {
            ok = false;                       // timed out (recorded): stop issuing, keep the warp converged
          } else {
            mbar_expect_tx(full0 + 8 * st, kAttTileBytes);
            tma_load_3d(ring0 + st * kAttTileBytes, &tmKV, full0 + 8 * st, 0, row, layer);
          }
        }
        if (++st == stages) { st = 0; ph ^= 1u; }
      }
      ++s;
    }
  } else if (warp == 5) {
    // ---- P V issuer (lane 0): O += P V as soon as the softmax threads have stored P; a segment's first product
    // overwrites the accumulator (the softmax threads read the previous segment's before they store these weights)
    if (lane == 0) {
      constexpr uint32_t idesc_pv = umma_idesc_bf16(128, 64) | (1u << 16);     // B (V tile) is MN-major
      bool ok = true;
      int g = 0;
      while (ok && it.next(sg)) {
        const int ntiles = sg.p1 - sg.p0;
        for (int i = 0; i < ntiles; ++i, ++g) {
          if (!mbar_wait(bar_p0 + 8 * (g % 3), (g / 3) & 1, err)) { ok = false; break; }
          if (!mbar_wait(full_v0 + 8 * (g % SV), (g / SV) & 1, err)) { ok = false; break; }
          tc_fence_after();
          const uint32_t va = ring_v + (g % SV) * kAttTileBytes, pa = tmem + 64 * (g % 3);
#pragma unroll
          for (int k = 0; k < 4; ++k)        // 16 keys per step: 8 TMEM columns of A, 16 rows (2048 bytes) of V
            umma_bf16_ts(tmem + 192, pa + 8 * k, umma_desc_k_sw128(va + 2048 * k), idesc_pv, (i | k) != 0);
#pragma unroll
          for (int k = 0; k < 4; ++k)        // the lo halves of the weights
            umma_bf16_ts(tmem + 192, pa + 32 + 8 * k, umma_desc_k_sw128(va + 2048 * k), idesc_pv, true);
          umma_commit(empty_v0 + 8 * (g % SV));
          umma_commit(bar_o0 + 8 * (g % 3));
        }
      }
    }
  } else if (warp == 6) {
    // ---- Q K^T issuer (lane 0): S = Q K^T into score buffer g % 3, up to three pages ahead of P V, also across
    // the end of a segment
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(128, 64);
      bool ok = true;
      int g = 0, s = 0;
      while (ok && it.next(sg)) {
        const int ntiles = sg.p1 - sg.p0;
        if (!mbar_wait(q_full0 + 8 * (s & 1), (s >> 1) & 1, err)) break;
        const uint32_t qa = q_addr + (s & 1) * kAsQBytes;
        for (int i = 0; i < ntiles; ++i, ++g) {
          // the buffer held the weights of page g - 3: free once that page's P V has completed
          if (g >= 3 && !mbar_wait(bar_o0 + 8 * (g % 3), ((g - 3) / 3) & 1, err)) { ok = false; break; }
          const int st = g % SK;
          if (!mbar_wait(full_k0 + 8 * st, (g / SK) & 1, err)) { ok = false; break; }
          tc_fence_after();
          const uint32_t ka = ring + st * kAttTileBytes;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16(tmem + 64 * (g % 3), umma_desc_k_sw128(qa + 32 * k), umma_desc_k_sw128(ka + 32 * k), idesc_qk, k != 0);
          umma_commit(empty_k0 + 8 * st);                    // the K tile is free once these MMAs have read it
          umma_commit(bar_s0 + 8 * (g % 3));
        }
        ++s;
      }
    }
  } else {
    // ---- softmax and epilogue: thread tid owns TMEM lane tid = query row (tid & 63), keys 32*half .. 32*half+31
    // of each page
    const int row = tid & 63, half = tid >> 6;
    const uint32_t trow = tmem + ((uint32_t)(32 * warp) << 16);
    auto wait_ok = [&](uint32_t bar, uint32_t parity) -> bool {
      if (*s_abort) return false;
      if (mbar_wait(bar, parity, err)) return true;
      *s_abort = 1;
      return false;
    };
    // sequences without a tree have no pages in the stream: their output rows are cleared here
    for (int b = c; b < batch; b += (int)gridDim.x)
      if ((meta[b] >> 24) == 0) {
        uint4* dst = reinterpret_cast<uint4*>(out + (long long)b * N * d_model);
        for (long long e = tid; e < (long long)N * d_model / 8; e += 128) dst[e] = make_uint4(0, 0, 0, 0);
      }
    bool has = it.next(sg);
    unsigned long long alo = 0ull, ahi = 0ull;                     // ancestor-or-self bits of this row's node
    if (has && row < (int)(meta[sg.b] >> 24)) tree.anc_of(sg.b, row, alo, ahi);
    int g = 0, s = 0;
    while (has) {
      const int b = sg.b, ntiles = sg.p1 - sg.p0;
      const int nv = (int)(meta[b] >> 24), ctx = (int)(meta[b] & 0xffffffu);
      const int total = ctx + nv;
      float m_use = -INFINITY, l_run = 0.f;       // scaling maximum (log2 units) and partial sum of this key half
      for (int i = 0; i < ntiles; ++i, ++g) {
        const int page = sg.p0 + i;
        wait_ok(bar_s0 + 8 * (g % 3), (g / 3) & 1);
        tc_fence_after();
        const uint32_t tsp = trow + 64 * (g % 3);       // this page's score / weight buffer
        float sc[32];
        tmem_ld32(tsp + 32 * half, sc);
        const int key0 = page * kKvBlock + 32 * half;
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
        for (int q = 0; q < 4; ++q) {
          mx4[q] = fmax3(sc[8 * q], sc[8 * q + 1], sc[8 * q + 2]);
          mx4[q] = fmax3(mx4[q], sc[8 * q + 3], sc[8 * q + 4]);
          mx4[q] = fmax3(mx4[q], sc[8 * q + 5], sc[8 * q + 6]);
          mx4[q] = fmaxf(mx4[q], sc[8 * q + 7]);
        }
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        if ((page + 1) * kKvBlock > total && tid < 64) {   // rows of V past the tree may hold anything: zero them
          const int valid = total - page * kKvBlock;
          wait_ok(full_v0 + 8 * (g % SV), (g / SV) & 1);             // the V tile has landed before rows of it are cleared
          if (tid >= valid) {
            uint4* vr = reinterpret_cast<uint4*>(ring_ptr + (SK + g % SV) * kAttTileBytes + tid * 128);
#pragma unroll
            for (int q = 0; q < 8; ++q) vr[q] = make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async_smem();
        }
        mx *= scale_log2e;                      // raw scores; the (positive) scale moves into the exponent
        // move the scaling maximum only when the page maximum exceeds it by more than the step
        float factor = 1.f;
        if (mx > m_use + kAttRescaleStep || m_use == -INFINITY) {
          factor = (m_use == -INFINITY) ? 0.f : fast_exp2(m_use - mx);
          if (mx > -INFINITY) m_use = mx;
        }
        if (i > 0 && __any_sync(0xffffffffu, factor != 1.f)) {
          // rescale this row's accumulator, once the previous page's P V has completed
          wait_ok(bar_o0 + 8 * ((g - 1) % 3), ((g - 1) / 3) & 1);
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
        mbar_arrive(bar_p0 + 8 * (g % 3));
      }
      // the next segment and its ancestor bits, fetched while the last P V of this one completes
      StreamSeg nx;
      const bool has_next = it.next(nx);
      unsigned long long nlo = 0ull, nhi = 0ull;
      if (has_next && row < (int)(meta[nx.b] >> 24)) tree.anc_of(nx.b, row, nlo, nhi);
      wait_ok(bar_o0 + 8 * ((g - 1) % 3), ((g - 1) / 3) & 1);
      tc_fence_after();

      // ---- epilogue of the segment: rows r and r + 64 are the two key halves of node r
      float* Ox = reinterpret_cast<float*>(base_ptr + (s & 1) * kAsQBytes);   // [64][64] fp32 over this segment's Q,
      float o_acc[64];                                                        // row r rotated by 4r columns
      tmem_ld32(trow + 192, o_acc);
      tmem_ld32(trow + 224, o_acc + 32);
      lx[tid] = l_run;
      lx[128 + tid] = m_use;
      if (tid >= 64) {
#pragma unroll
        for (int e = 0; e < 64; ++e) Ox[(tid - 64) * 64 + ((e + 4 * tid) & 63)] = o_acc[e];
      }
      as_bar128(1);
      if (tid < 64) {
        // the two key halves of the row on a common scale
        const float m1 = lx[128 + tid + 64], mm = fmaxf(m_use, m1);
        const float w0 = (m_use == -INFINITY) ? 0.f : fast_exp2(m_use - mm), w1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - mm);
#pragma unroll
        for (int e = 0; e < 64; ++e) o_acc[e] = o_acc[e] * w0 + Ox[tid * 64 + ((e + 4 * tid) & 63)] * w1;
        l_run = l_run * w0 + lx[tid + 64] * w1;
        m_use = mm;
        if (sg.parts == 1) {
          if (tid < N) {
            const float inv = (tid < nv && l_run > 0.f) ? 1.f / l_run : 0.f;
            uint4* dst = reinterpret_cast<uint4*>(out + ((long long)b * N + tid) * d_model + h * 64);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              uint4 v;
              v.x = pack_bf16(o_acc[8 * q + 0] * inv, o_acc[8 * q + 1] * inv);
              v.y = pack_bf16(o_acc[8 * q + 2] * inv, o_acc[8 * q + 3] * inv);
              v.z = pack_bf16(o_acc[8 * q + 4] * inv, o_acc[8 * q + 5] * inv);
              v.w = pack_bf16(o_acc[8 * q + 6] * inv, o_acc[8 * q + 7] * inv);
              dst[q] = v;
            }
          }
        } else {
          // this part's (O, l, m) goes to the CTA's first or second exchange slot (it stays in L2)
          float* mine = xch + (long long)(2 * c + (sg.first_of_cta ? 0 : 1)) * kAsSlotFloats;
          float4* dst = reinterpret_cast<float4*>(mine + tid * 64);
#pragma unroll
          for (int q = 0; q < 16; ++q) dst[q] = make_float4(o_acc[4 * q], o_acc[4 * q + 1], o_acc[4 * q + 2], o_acc[4 * q + 3]);
          mine[64 * 64 + tid] = l_run;
          mine[64 * 64 + 64 + tid] = m_use;
          __threadfence();
        }
      }
      as_bar128(1);                            // the exchange over Q has been read; the part's slot is written
      if (tid == 0) {
        fence_proxy_async_smem();              // the next Q into this buffer is written by the TMA unit
        mbar_arrive(q_empty0 + 8 * (s & 1));
      }
      if (sg.parts > 1) {
        // slot of part 0: its CTA's first segment or its last; later parts are their CTAs' first segments
        const int slot0 = 2 * (sg.first_grp * H + h) + (sg.part0_first ? 0 : 1);
        if (tid == 0) {
          // the part that arrives last merges; the counter is left at zero for the next launch
          const uint32_t old = atomicAdd(cnt + slot0, 1u);
          const int last = old == (uint32_t)(sg.parts - 1);
          if (last) cnt[slot0] = 0u;
          __threadfence();
          *s_flag = last;
        }
        as_bar128(1);
        if (*s_flag) {
          // thread = (node, half of the features); the parts in their order along the sequence, whichever arrived
          // last; every part's loads are independent of one another (one L2 round trip per part)
          const int r = tid & 63, ch = tid >> 6;
          float M = -INFINITY;
          for (int q = 0; q < sg.parts; ++q) {
            const float* sl = xch + (long long)(q == 0 ? slot0 : 2 * ((sg.first_grp + q) * H + h)) * kAsSlotFloats;
            M = fmaxf(M, __ldcg(sl + 64 * 64 + 64 + r));
          }
          float L = 0.f;
          float acc[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) acc[e] = 0.f;
#pragma unroll 2
          for (int q = 0; q < sg.parts; ++q) {
            const float* sl = xch + (long long)(q == 0 ? slot0 : 2 * ((sg.first_grp + q) * H + h)) * kAsSlotFloats;
            const float mq = __ldcg(sl + 64 * 64 + 64 + r), lq = __ldcg(sl + 64 * 64 + r);
            const float4* src = reinterpret_cast<const float4*>(sl + r * 64 + 32 * ch);
            float4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __ldcg(src + j);
            const float w = (mq == -INFINITY) ? 0.f : exp2f(mq - M);
            L = fmaf(lq, w, L);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              acc[4 * j + 0] = fmaf(v[j].x, w, acc[4 * j + 0]); acc[4 * j + 1] = fmaf(v[j].y, w, acc[4 * j + 1]);
              acc[4 * j + 2] = fmaf(v[j].z, w, acc[4 * j + 2]); acc[4 * j + 3] = fmaf(v[j].w, w, acc[4 * j + 3]);
            }
          }
          if (r < N) {
            const float inv = (r < nv && L > 0.f) ? 1.f / L : 0.f;
            uint4* dst = reinterpret_cast<uint4*>(out + ((long long)b * N + r) * d_model + h * 64 + 32 * ch);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint4 o;
              o.x = pack_bf16(acc[8 * j + 0] * inv, acc[8 * j + 1] * inv);
              o.y = pack_bf16(acc[8 * j + 2] * inv, acc[8 * j + 3] * inv);
              o.z = pack_bf16(acc[8 * j + 4] * inv, acc[8 * j + 5] * inv);
              o.w = pack_bf16(acc[8 * j + 6] * inv, acc[8 * j + 7] * inv);
              dst[j] = o;
            }
          }
        }
      }
      has = has_next;
      sg = nx;
      alo = nlo; ahi = nhi;
      ++s;
    }
  }
  __syncwarp();
  grid_dep_launch();
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 256);
}

}  // namespace vadusa
