// One persistent kernel for the whole verify pass of a single sequence (bf16, head_dim 64, at most 64
// tree nodes): embedding, every layer (LayerNorm -> q/k/v -> tree attention -> output projection ->
// LayerNorm -> feed-forward) and the final LayerNorm + vocabulary head, without a kernel boundary.
//
// Why: with one sequence a pass is a chain of dependent steps that each stream a few MB of weights; as
// separate kernels every step pays a launch hand-over, a cold start of its weight stream and an exchange
// through L2.  Here the grid is resident for the whole pass, weights and context K/V run ahead of the
// dependency chain through a TMA ring, and partial results are exchanged inside thread-block clusters
// through distributed shared memory.
//
// Grid: n_heads clusters of CS CTAs (CS = 8, or 6 where the device cannot hold n_heads clusters of 8 at once),
// one CTA per SM.  Cluster c owns head c (q/k/v rows of head c and its
// attention), rows [64c, 64c+64) of the output projection and of the second feed-forward matrix, rows
// [c F/H, (c+1) F/H) of the first one, and vocabulary tiles c, c+H, ...  Inside a cluster CTA r owns K slice
// r of every product (the 64-column chunks of the inner dimension are dealt out as evenly as CS allows) and
// context pages [r per, (r+1) per) of the attention.  Every product is computed as D[token][feature] = X[token][k] W[feature][k]^T with the tokens as
// the MMA's 128-row operand (64 tokens, stored twice where the epilogue is wide) and the CTA's weight rows as
// the narrow operand.  A product's K-slice partials are summed by the cluster: CTA r receives, from all CTAs
// of the cluster, the partial rows of its share of the tokens in its shared memory, adds them in a fixed order, applies the
// epilogue (bias, residual, ReLU, LayerNorm statistics) and publishes the result.
//
// Exchanges between clusters go through global memory (L2) with monotonic counters: producers store, fence
// and add to a counter with release semantics; consumers poll the counter with acquire loads.  Exchanges
// inside a cluster are remote shared-memory stores followed by a remote mbarrier arrival.
//
// Warps: 0 = TMA producer (one lane), 1 = MMA issuer (one lane) and TMEM owner, 2..5 = workers (operand
// construction, epilogues, softmax).  Every wait is bounded in time; a wait that runs out records
// kErrTimeout, sets the CTA's abort flag and every later wait returns at once, so the kernel always ends.
#pragma once
#include "attention_tc.cuh"
#include "tc.cuh"

namespace vadusa {

constexpr int kFfThreads = 192;
constexpr int kFfWorkers = 128;
constexpr uint32_t kFfSlotBytes = 16384;       // ring slot
constexpr uint32_t kFfTileBytes = 8192;        // 64 rows of 128 bytes
constexpr uint32_t kFfMiscBytes = 1024;
constexpr int kFfMaxPages = 32;                // context pages per CTA
constexpr int kFfGroup = 3;                    // pages per softmax group (three score buffers)
constexpr unsigned long long kFfWaitNs = 400ull * 1000 * 1000;

// Shared-memory plan for a cluster of CS CTAs (d_model <= 1024: at most 16 chunks of 64 columns).
template <int CS> struct FfCfg {
  static constexpr int kTpo = (64 + CS - 1) / CS;                       // tokens per owner, at most
  static constexpr int kMaxKc = (16 + CS - 1) / CS;                     // chunks of a CTA's K slice of d_model, at most
  static constexpr int kSlots = CS >= 8 ? 7 : 6;                        // ring slots
  static constexpr uint32_t kRingBytes = kSlots * kFfSlotBytes;
  // LayerNorm operand: one 128-row tile (16 KB) per chunk; also the Q tile + the tree's K and V tiles (32 KB)
  static constexpr uint32_t kXaBytes = kMaxKc * 16384u < 32768u ? 32768u : kMaxKc * 16384u;
  static constexpr uint32_t kRbBytes = 64 * (256 + 4) * 4;              // this CTA's K-slice partial [64 tokens][N + 4], read by the owners
  static constexpr uint32_t kQoBytes = ((kTpo * 192 * 2 + 1023) / 1024) * 1024;   // q/k/v rows of the owned tokens, read by the peers
  static constexpr int kSmemBytes = (int)(kRingBytes + kXaBytes + kRbBytes + kQoBytes + kFfMiscBytes + 1024 /*alignment*/);
  static constexpr int kRounds = (kTpo * 16 + kFfWorkers - 1) / kFfWorkers;   // passes of 128 threads over (token, 4 features)
};

constexpr uint32_t kFfColAcc = 0;              // TMEM columns: product accumulator (up to 256 features)
constexpr uint32_t kFfColS = 256;              // three score / weight buffers of 64 columns
constexpr uint32_t kFfColO = 448;              // attention output accumulator

// words of the synchronisation area (uint32): two counters, the pass counter, one word per head for the
// attention outputs and one per cluster for the feed-forward hidden layer
constexpr int kFfSyncXa = 0, kFfSyncXb = 1, kFfSyncDone = 2, kFfSyncO = 16, kFfSyncMid = 32, kFfSyncWords = 64;

// Items [first, first + count) of `total` dealt to part r of `parts` (the first total % parts parts get one more).
__host__ __device__ __forceinline__ void ff_split(int total, int parts, int r, int& first, int& count) {
  const int base = total / parts, rem = total % parts;
  count = base + (r < rem ? 1 : 0);
  first = r * base + (r < rem ? r : rem);
}
__host__ __device__ __forceinline__ int ff_owner(int item, int total, int parts) {
  const int base = total / parts, rem = total % parts, edge = rem * (base + 1);
  return item < edge ? item / (base + 1) : rem + (item - edge) / base;
}

struct FusedArgs {
  int L, d, H, F, vocab, vpad, n_phonemes, max_pos, M;
  float eps, scale_log2e;
  const float *ln1_g, *ln1_b, *bqkv, *bo, *ln2_g, *ln2_b, *b1, *b2;     // layer 0; later layers at a constant stride
  long long layer_stride;          // bytes between the same tensor of consecutive layers
  const float *lnf_g, *lnf_b;
  const bf16 *emb_audio, *emb_phon, *pos;
  float *xa, *xb;                  // fp32 residual stream: layer input / after the attention block  [M][d]
  float2 *stats_a, *stats_b;       // [M][H]: mean and sum of squared deviations of each group of 64 features
  bf16 *o, *mid, *hfinal;          // [M][d], [M][F], [M][d]
  float* logits;                   // [M][vpad]
  bf16* attn_tap;                  // [L][M][d] or null
  int32_t* tokens;                 // [M]
  long long* kv_row;               // [M]
  const int32_t *override_tokens, *root, *topk;
  int n_draft_heads, draft_topk;
  const int32_t *ctx_len, *nvalid, *block_table;
  TreeView tree;
  KvGeom geom;
  bf16* kv_pool;
  uint32_t* sync;
  uint32_t* err;
};

// ---- small PTX helpers -----------------------------------------------------------------
__device__ __forceinline__ unsigned long long ff_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ uint32_t ff_ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ff_ld_relaxed(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void ff_red_release(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ff_mapa(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  return remote;
}
__device__ __forceinline__ void ff_st_cluster_f4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void ff_st_cluster_u4(uint32_t addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float4 ff_ld_cluster_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ff_ld_cluster_u4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared::cluster.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void ff_st_shared_f4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void ff_st_shared_u4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void ff_arrive_remote(uint32_t remote_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ bool ff_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void ff_fence_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
__device__ __forceinline__ void ff_fence_proxy_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void ff_fence_proxy_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void ff_workers_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Bounded wait: polls `ready` until it holds, the CTA's abort flag is up, the device error word carries
// a timeout from anywhere in the grid, or the time limit passes (then records the timeout).
template <typename F>
__device__ __forceinline__ bool ff_wait(F&& ready, uint32_t* err, volatile int* abort_flag) {
  if (*abort_flag) return false;
  if (ready()) return true;
  const unsigned long long t0 = ff_timer();
  for (uint32_t i = 1;; ++i) {
    if (ready()) return true;
    if ((i & 63u) == 0u) {
      if (*abort_flag) return false;
      const bool late = ff_timer() - t0 > kFfWaitNs;
      if (late || (ff_ld_relaxed(err) & kErrTimeout)) {
        if (late) atomicOr(err, kErrTimeout);
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ uint4 ff_pack8(const float* v) {
  uint4 r;
  r.x = pack_bf16(v[0], v[1]); r.y = pack_bf16(v[2], v[3]); r.z = pack_bf16(v[4], v[5]); r.w = pack_bf16(v[6], v[7]);
  return r;
}


template <int CS>
__global__ void __launch_bounds__(kFfThreads, 1) fused_forward_kernel(
    const __grid_constant__ CUtensorMap tmQkv,   // [L][3d][d]    box 64 rows x 64
    const __grid_constant__ CUtensorMap tmWo,    // [L][d][d]     box 64 x 64
    const __grid_constant__ CUtensorMap tmW1,    // [L][F][d]     box 128 x 64
    const __grid_constant__ CUtensorMap tmW2,    // [L][d][F]     box 64 x 64
    const __grid_constant__ CUtensorMap tmLm,    // [1][vpad][d]  box 128 x 64
    const __grid_constant__ CUtensorMap tmO,     // [1][M][d]     box 64 x 64
    const __grid_constant__ CUtensorMap tmMid,   // [1][M][F]     box 64 x 64
    const __grid_constant__ CUtensorMap tmKV,    // [L][blocks * 2 * H * 64][64]  box 64 x 64
    const FusedArgs a) {
  using Cfg = FfCfg<CS>;
  constexpr int R = Cfg::kSlots, KCMAX = Cfg::kMaxKc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_p = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t ring = base, xa = base + Cfg::kRingBytes, rb = xa + Cfg::kXaBytes, qo = rb + Cfg::kRbBytes, bars = qo + Cfg::kQoBytes;
  uint8_t* ring_p = base_p;
  uint8_t* misc_p = base_p + Cfg::kRingBytes + Cfg::kXaBytes + Cfg::kRbBytes + Cfg::kQoBytes;
  const uint32_t full0 = bars, empty0 = bars + 64, bar_xa = bars + 128, bar_acc = bars + 136, bar_accfree = bars + 144,
                 bar_s = bars + 152, bar_p = bars + 160, bar_o = bars + 168, bar_qkv = bars + 176,
                 bar_rbfull = bars + 184, bar_rbfree = bars + 192, holder = bars + 200, bar_q = bars + 208;
  volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(misc_p + 200);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc_p + 204);
  float2* s_rowstat = reinterpret_cast<float2*>(misc_p + 256);         // [64] (mean, rstd)
  int* s_pageblk = reinterpret_cast<int*>(misc_p + 768);               // [kFfMaxPages] pool row of each of this CTA's pages
  long long* s_kvrow = reinterpret_cast<long long*>(misc_p + 896);     // [TPO] K slot of this CTA's tokens (head 0), or -1

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = (int)cluster_rank();
  const int c = (int)blockIdx.x / CS;                    // cluster = head
  const int NC = (int)gridDim.x / CS;
  const int G = (int)gridDim.x;
  const int d = a.d, F = a.F, L = a.L, M = a.M;
  int kc0, nkc, kf0, nk2;                                // this CTA's 64-column chunks of d_model and of the feed-forward width
  ff_split(d / 64, CS, rank, kc0, nkc);
  ff_split(F / 64, CS, rank, kf0, nk2);
  const int n1 = F / NC, nrb = n1 / 128;                 // rows of the first feed-forward matrix per cluster, in blocks of 128
  const int nlm = a.vpad / 128;                          // vocabulary tiles
  const int npair = (nkc + 1) / 2;                       // ring items of a list of nkc 8 KB tiles (two per item)
  uint32_t* err = a.err;

  if (tid == 0) {
    for (int s = 0; s < R; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(bar_xa, kFfWorkers); mbar_init(bar_acc, 1); mbar_init(bar_accfree, kFfWorkers);
    mbar_init(bar_s, 1); mbar_init(bar_p, kFfWorkers); mbar_init(bar_o, 1);
    mbar_init(bar_qkv, 4 * CS); mbar_init(bar_rbfull, 4 * CS); mbar_init(bar_rbfree, CS); mbar_init(bar_q, kFfWorkers);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQkv); tma_prefetch_desc(&tmWo); tma_prefetch_desc(&tmW1); tma_prefetch_desc(&tmW2);
    tma_prefetch_desc(&tmLm); tma_prefetch_desc(&tmO); tma_prefetch_desc(&tmMid); tma_prefetch_desc(&tmKV);
  }
  // the operand area starts out finite (rows of it that no one writes are read by MMAs whose results are unused,
  // and as keys / values with zero weight)
  for (int i = tid; i < (int)(Cfg::kXaBytes / 16); i += kFfThreads) reinterpret_cast<uint4*>(base_p + Cfg::kRingBytes)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 1) { tmem_alloc(holder, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                           // the peers' barriers are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem = *holder_ptr;

  // Per-layer ring items, numbered in issue order (the same arithmetic in every role):
  //   offQK + kc       q rows | k rows of head c, chunk kc
  //   offV + kc/2      v rows, chunks kc (two tiles per item)
  //   offKV + i        context page i of this CTA (K tile | V tile)
  //   offOutW + kc/2   output-projection rows [64c, 64c+64), chunks kc
  //   offOutX + kc/2   attention output (tokens), chunks kc; waits for the heads that make those columns
  //   offF1 + rb*nkc + kc   rows 128 rb .. of the first feed-forward matrix, chunk kc
  //   offF2 + j        chunk j of: hidden activations (tokens) | rows of the second feed-forward matrix
  // The first feed-forward matrix is issued ahead of the (gated) attention output when the ring has room for both.
  int ctx = 0, nv = 0, np_mine = 0, p0 = 0;
  int offV = 0, offKV = 0, offOutW = 0, offOutX = 0, offF1 = 0, offF2 = 0, ipl = 0;
  bool f1_first = false;
  auto plan = [&]() {                           // after griddepcontrol.wait
    ctx = a.ctx_len[0]; nv = a.nvalid[0];
    const int npages = nv > 0 ? (ctx + kKvBlock - 1) / kKvBlock : 0;
    const int per = (npages + CS - 1) / CS;
    p0 = rank * per;
    const int p1 = min(npages, p0 + per);
    np_mine = max(0, p1 - p0);
    if (np_mine > kFfMaxPages) { np_mine = kFfMaxPages; atomicOr(err, kErrCapacity); }
    const int nf1 = nrb * nkc;
    offV = nkc; offKV = offV + npair; offOutW = offKV + np_mine;
    f1_first = npair + nf1 + npair - 1 < R;
    if (f1_first) { offF1 = offOutW + npair; offOutX = offF1 + nf1; offF2 = offOutX + npair; }
    else { offOutX = offOutW + npair; offF1 = offOutX + npair; offF2 = offF1 + nf1; }
    ipl = offF2 + nk2;
  };
  const bool lm_mine = c < nlm;

  if (warp == 0) {
    // =========================================================== TMA producer
    grid_dep_wait();
    plan();
    if (lane < np_mine) {
      const long long blk = kv_block_of(a.block_table, a.geom, 0, (p0 + lane) * kKvBlock, err);
      s_pageblk[lane] = (int)((blk < 0 ? 0 : blk) * 2 * a.geom.n_heads + c) * kKvBlock;
    }
    __syncwarp();
    if (lane == 0) {
      bool ok = true;
      // slot of item `seq`: waits until the item that used it before has been consumed; arms the barrier
      auto acquire = [&](int seq, uint32_t bytes) -> uint32_t {
        const int s = seq % R;
        if (seq >= R)
          ok = ok && ff_wait([&] { return mbar_try_wait(empty0 + 8 * s, ((seq / R) - 1) & 1); }, err, abort_flag);
        if (ok) mbar_expect_tx(full0 + 8 * s, bytes);
        return ring + s * kFfSlotBytes;
      };
      auto fullbar = [&](int seq) -> uint32_t { return full0 + 8 * (seq % R); };
      auto gate = [&](int word, uint32_t target) {
        ok = ok && ff_wait([&] { return ff_ld_acquire(a.sync + word) >= target; }, err, abort_flag);
      };
      // a list of nkc tiles (64 rows x chunk kc of `map` at row `row`), two per item
      auto issue_pairs = [&](int seq0, const CUtensorMap* map, int row, int z) {
        for (int i = 0; i < npair && ok; ++i) {
          const int nt = min(2, nkc - 2 * i);
          const uint32_t dst = acquire(seq0 + i, nt * kFfTileBytes);
          if (!ok) break;
          for (int t = 0; t < nt; ++t) tma_load_3d(dst + t * kFfTileBytes, map, fullbar(seq0 + i), 64 * (kc0 + 2 * i + t), row, z);
        }
      };
      for (int l = 0; l < L && ok; ++l) {
        const int b0 = l * ipl;
        for (int kc = 0; kc < nkc && ok; ++kc) {
          const uint32_t dst = acquire(b0 + kc, 2 * kFfTileBytes);
          if (!ok) break;
          tma_load_3d(dst, &tmQkv, fullbar(b0 + kc), 64 * (kc0 + kc), c * 64, l);
          tma_load_3d(dst + kFfTileBytes, &tmQkv, fullbar(b0 + kc), 64 * (kc0 + kc), d + c * 64, l);
        }
        issue_pairs(b0 + offV, &tmQkv, 2 * d + c * 64, l);
        for (int i = 0; i < np_mine && ok; ++i) {
          const uint32_t dst = acquire(b0 + offKV + i, 2 * kFfTileBytes);
          if (!ok) break;
          tma_load_3d(dst, &tmKV, fullbar(b0 + offKV + i), 0, s_pageblk[i], l);
          tma_load_3d(dst + kFfTileBytes, &tmKV, fullbar(b0 + offKV + i), 0, s_pageblk[i] + a.geom.n_heads * kKvBlock, l);
        }
        issue_pairs(b0 + offOutW, &tmWo, c * 64, l);
        auto issue_f1 = [&]() {
          for (int i = 0; i < nrb * nkc && ok; ++i) {
            const uint32_t dst = acquire(b0 + offF1 + i, 2 * kFfTileBytes);
            if (!ok) break;
            tma_load_3d(dst, &tmW1, fullbar(b0 + offF1 + i), 64 * (kc0 + i % nkc), c * n1 + 128 * (i / nkc), l);
          }
        };
        auto issue_outx = [&]() {
          // every head whose 64 output columns lie in this K slice has published them
          for (int kc = 0; kc < nkc; ++kc) gate(kFfSyncO + kc0 + kc, (uint32_t)(CS * (l + 1)));
          ff_fence_proxy_global();
          issue_pairs(b0 + offOutX, &tmO, 0, 0);
        };
        if (f1_first) { issue_f1(); issue_outx(); } else { issue_outx(); issue_f1(); }
        // second feed-forward matrix: weight tiles first, as far as the ring goes (they stream while the hidden
        // layer is computed), then the hidden activations once every cluster that makes this K slice has
        // published them; the rest in pairs as slots come free
        const int nw = min(nk2, R);
        for (int j = 0; j < nw && ok; ++j) {
          const uint32_t dst = acquire(b0 + offF2 + j, 2 * kFfTileBytes);
          if (!ok) break;
          tma_load_3d(dst + kFfTileBytes, &tmW2, fullbar(b0 + offF2 + j), 64 * (kf0 + j), c * 64, l);
        }
        if (nk2 > 0)
          for (int cc = (64 * kf0) / n1; cc <= (64 * (kf0 + nk2) - 1) / n1; ++cc) gate(kFfSyncMid + cc, (uint32_t)(CS * (l + 1)));
        ff_fence_proxy_global();
        for (int j = 0; j < nw && ok; ++j)
          tma_load_3d(ring + ((b0 + offF2 + j) % R) * kFfSlotBytes, &tmMid, fullbar(b0 + offF2 + j), 64 * (kf0 + j), 0, 0);
        for (int j = nw; j < nk2 && ok; ++j) {
          const uint32_t dst = acquire(b0 + offF2 + j, 2 * kFfTileBytes);
          if (!ok) break;
          tma_load_3d(dst + kFfTileBytes, &tmW2, fullbar(b0 + offF2 + j), 64 * (kf0 + j), c * 64, l);
          tma_load_3d(dst, &tmMid, fullbar(b0 + offF2 + j), 64 * (kf0 + j), 0, 0);
        }
      }
      if (lm_mine) {
        int seq = L * ipl;
        for (int t = c; t < nlm && ok; t += NC)
          for (int kc = 0; kc < nkc && ok; ++kc, ++seq) {
            const uint32_t dst = acquire(seq, 2 * kFfTileBytes);
            if (!ok) break;
            tma_load_3d(dst, &tmLm, fullbar(seq), 64 * (kc0 + kc), 128 * t, 0);
          }
      }
    }
  }
  else if (warp == 1) {
    // =========================================================== MMA issuer
    grid_dep_wait();
    plan();
    if (lane == 0) {
      constexpr uint32_t id128 = umma_idesc_bf16(128, 128), id64 = umma_idesc_bf16(128, 64);
      constexpr uint32_t id_pv = umma_idesc_bf16(128, 64) | (1u << 16);        // B (V tile) is MN-major
      const uint32_t acc = tmem + kFfColAcc;
      bool ok = true;
      uint32_t n_xa = 0, n_accfree = 0, n_p = 0, n_qkv = 0;
      bool first_acc = true;
      auto wait_full = [&](int seq) -> uint32_t {
        const int s = seq % R;
        ok = ok && ff_wait([&] { return mbar_try_wait(full0 + 8 * s, (seq / R) & 1); }, err, abort_flag);
        return ring + s * kFfSlotBytes;
      };
      auto release = [&](int seq) { umma_commit(empty0 + 8 * (seq % R)); };
      auto wait_local = [&](uint32_t bar, uint32_t& n) {
        ok = ok && ff_wait([&] { return mbar_try_wait(bar, n & 1); }, err, abort_flag);
        ++n;
      };
      // the workers have read the previous product's accumulator
      auto acc_begin = [&]() {
        if (!first_acc) wait_local(bar_accfree, n_accfree);
        first_acc = false;
        tc_fence_after();
      };
      // four K steps of 16: D (+)= A[128 x 64] B[N x 64]^T
      auto mma4 = [&](uint32_t dcol, uint32_t a_addr, uint32_t b_addr, uint32_t idesc, bool accumulate) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(dcol, umma_desc_k_sw128(a_addr + 32 * k), umma_desc_k_sw128(b_addr + 32 * k), idesc, accumulate || k != 0);
      };
      const int ntile = np_mine + ((rank == CS - 1 && nv > 0) ? 1 : 0);
      for (int l = 0; l < L && ok; ++l) {
        const int b0 = l * ipl;
        // ---- q/k/v: D[:, 0:64) = q, [64:128) = k, [128:192) = v
        acc_begin();
        wait_local(bar_xa, n_xa);
        tc_fence_after();
        for (int kc = 0; kc < nkc && ok; ++kc) {
          const uint32_t w = wait_full(b0 + kc);
          if (!ok) break;
          tc_fence_after();
          mma4(acc, xa + kc * 16384, w, id128, kc != 0);
          release(b0 + kc);
        }
        for (int kc = 0; kc < nkc && ok; ++kc) {
          const uint32_t w = wait_full(b0 + offV + kc / 2);
          if (!ok) break;
          tc_fence_after();
          mma4(acc + 128, xa + kc * 16384, w + (kc & 1) * kFfTileBytes, id64, kc != 0);
          if ((kc & 1) || kc == nkc - 1) release(b0 + offV + kc / 2);
        }
        if (!ok) break;
        umma_commit(bar_acc);
        // ---- attention of head c over this CTA's pages (and the tree's own keys in the last CTA)
        wait_local(bar_q, n_qkv);               // the workers have gathered the Q tile (and the tree's K, V tiles)
        tc_fence_after();
        for (int t0 = 0; t0 < ntile && ok; t0 += kFfGroup) {
          const int npg = min(kFfGroup, ntile - t0);
          for (int pi = 0; pi < npg && ok; ++pi) {
            const int t = t0 + pi;
            const uint32_t ka = t < np_mine ? wait_full(b0 + offKV + t) : xa + 16384;
            if (!ok) break;
            tc_fence_after();
            mma4(tmem + kFfColS + 64 * pi, xa, ka, id64, false);
          }
          if (!ok) break;
          umma_commit(bar_s);
          wait_local(bar_p, n_p);
          if (!ok) break;
          tc_fence_after();
          for (int pi = 0; pi < npg; ++pi) {
            const int t = t0 + pi;
            const uint32_t va = t < np_mine ? ring + ((b0 + offKV + t) % R) * kFfSlotBytes + kFfTileBytes : xa + 24576;
            const uint32_t pa = tmem + kFfColS + 64 * pi;
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_bf16_ts(tmem + kFfColO, pa + 8 * k, umma_desc_k_sw128(va + 2048 * k), id_pv, (t | k) != 0);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_bf16_ts(tmem + kFfColO, pa + 32 + 8 * k, umma_desc_k_sw128(va + 2048 * k), id_pv, true);
            if (t < np_mine) release(b0 + offKV + t);
          }
          umma_commit(bar_o);
        }
        if (!ok) break;
        // ---- output projection
        acc_begin();
        for (int kc = 0; kc < nkc && ok; ++kc) {
          const uint32_t w = wait_full(b0 + offOutW + kc / 2);
          const uint32_t x = wait_full(b0 + offOutX + kc / 2);
          if (!ok) break;
          tc_fence_after();
          mma4(acc, x + (kc & 1) * kFfTileBytes, w + (kc & 1) * kFfTileBytes, id64, kc != 0);
          if ((kc & 1) || kc == nkc - 1) { release(b0 + offOutW + kc / 2); release(b0 + offOutX + kc / 2); }
        }
        if (!ok) break;
        umma_commit(bar_acc);
        // ---- first feed-forward matrix
        acc_begin();
        wait_local(bar_xa, n_xa);
        tc_fence_after();
        for (int i = 0; i < nrb * nkc && ok; ++i) {
          const uint32_t w = wait_full(b0 + offF1 + i);
          if (!ok) break;
          tc_fence_after();
          const int kc = i % nkc, rbk = i / nkc;
          mma4(acc + 128 * rbk, xa + kc * 16384, w, id128, kc != 0);
          release(b0 + offF1 + i);
        }
        if (!ok) break;
        umma_commit(bar_acc);
        // ---- second feed-forward matrix
        acc_begin();
        for (int j = 0; j < nk2 && ok; ++j) {
          const uint32_t s = wait_full(b0 + offF2 + j);
          if (!ok) break;
          tc_fence_after();
          mma4(acc, s, s + kFfTileBytes, id64, j != 0);
          release(b0 + offF2 + j);
        }
        if (!ok) break;
        umma_commit(bar_acc);
      }
      // ---- vocabulary head
      if (lm_mine && ok) {
        int seq = L * ipl;
        bool first = true;
        for (int t = c; t < nlm && ok; t += NC) {
          acc_begin();
          if (first) { wait_local(bar_xa, n_xa); first = false; tc_fence_after(); }
          for (int kc = 0; kc < nkc && ok; ++kc, ++seq) {
            const uint32_t w = wait_full(seq);
            if (!ok) break;
            tc_fence_after();
            mma4(acc, xa + kc * 16384, w, id128, kc != 0);
            release(seq);
          }
          if (ok) umma_commit(bar_acc);
        }
      }
    }
  }
  else {
    // =========================================================== workers (128 threads)
    const int wtid = tid - 64, ww = warp - 2, wq = warp & 3;
    const int lane_t = 32 * wq + lane;                       // this thread's TMEM lane
    const int tok_t = lane_t & 63, half_t = lane_t >> 6;     // token of the lane, which copy of it
    int tok0, ntok;                                          // the tokens this CTA owns
    ff_split(64, CS, rank, tok0, ntok);
    const uint32_t trow = tmem + ((uint32_t)(32 * wq) << 16);
    uint32_t n_acc = 0, n_rb = 0, n_s = 0, n_o = 0, n_qkv = 0;
    const long long kv_stride = (long long)a.geom.n_heads * kKvBlock * a.geom.head_dim;   // K row -> V row of a head
    const int tile_elems = kKvBlock * a.geom.head_dim;

    auto wait_bar = [&](uint32_t bar, uint32_t& n) {
      ff_wait([&] { return mbar_try_wait(bar, n & 1); }, err, abort_flag);
      ++n;
    };
    auto wait_counter = [&](int word, uint32_t target) {     // one poller, then the workers' barrier
      if (wtid == 0) ff_wait([&] { return ff_ld_acquire(a.sync + word) >= target; }, err, abort_flag);
      ff_workers_sync();
    };
    // every worker has stored its part; tma: the data is read by TMA loads (async proxy) of other CTAs
    auto publish = [&](int word, bool tma) {
      if (tma) ff_fence_proxy_global();
      ff_workers_sync();
      if (wtid == 0) { __threadfence(); ff_red_release(a.sync + word, 1u); }
    };
    // the receive buffers of the cluster are free again (every peer has read what the last round left)
    auto rb_begin = [&]() {
      if (n_rb > 0) ff_wait([&] { return ff_try_wait_cluster(bar_rbfree, (n_rb - 1) & 1); }, err, abort_flag);
    };
    auto rb_sent = [&]() {                                   // after this warp's remote stores
      ff_fence_cluster();
      __syncwarp();
      if (lane == 0)
        for (uint32_t p = 0; p < (uint32_t)CS; ++p) ff_arrive_remote(ff_mapa(bar_rbfull, p));
    };
    auto rb_wait = [&]() {
      ff_wait([&] { return ff_try_wait_cluster(bar_rbfull, n_rb & 1); }, err, abort_flag);
    };
    auto rb_done = [&]() {                                   // after this CTA's reads of its receive buffer
      ff_workers_sync();
      if (wtid == 0)
        for (uint32_t p = 0; p < (uint32_t)CS; ++p) ff_arrive_remote(ff_mapa(bar_rbfree, p));
      ++n_rb;
    };
    // K-slice partial D[token][0:N) of this CTA -> its own shared memory as [token][N + 4] fp32 (rows padded by 16
    // bytes: the lanes of a warp, one token each, then fall into different banks); the owners of the tokens read it
    // from there.  dup: tokens are stored twice in the operand, the second copy's lanes take the upper half of the
    // columns; else lanes 0..63 store everything.
    auto send_partial = [&](int N, bool dup) {
      wait_bar(bar_acc, n_acc);
      tc_fence_after();
      rb_begin();
      const int ncol = dup ? N / 2 : (half_t == 0 ? N : 0), col0 = dup ? half_t * (N / 2) : 0;
      const uint32_t dst = rb + (uint32_t)(tok_t * (N + 4) + col0) * 4u;
      for (int c0 = 0; c0 < ncol; c0 += 32) {                // (ncol is the same in all lanes of a warp)
        float v[32];
        tmem_ld32(trow + kFfColAcc + col0 + c0, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) ff_st_shared_f4(dst + (uint32_t)(c0 + 4 * i) * 4u, v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
      }
      rb_sent();
      tc_fence_before();
      mbar_arrive(bar_accfree);
    };
    // Sum over the CTAs of the cluster (fixed order) of four consecutive columns of one of this CTA's tokens.
    auto rb_sum4 = [&](int N, int tl, int col) -> float4 {
      const uint32_t off = rb + (uint32_t)((tok0 + tl) * (N + 4) + col) * 4u;
      float4 v[CS];
#pragma unroll
      for (int src = 0; src < CS; ++src) v[src] = ff_ld_cluster_f4(ff_mapa(off, (uint32_t)src));
      float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int src = 0; src < CS; ++src) { s.x += v[src].x; s.y += v[src].y; s.z += v[src].z; s.w += v[src].w; }
      return s;
    };
    // LayerNorm of this CTA's K-slice columns of rows x[0:M) into the operand tiles (each row stored at r and
    // r + 64).  Waits for `word` >= target first.  y: where to also store the normalised slice (or null).
    auto build_ln = [&](const float* x, const float2* stats, const float* g, const float* bta, int word, uint32_t target, bf16* y) {
      float4 gg[KCMAX], bb[KCMAX];
#pragma unroll
      for (int kc = 0; kc < KCMAX; ++kc)
        if (kc < nkc) {
          gg[kc] = __ldg(reinterpret_cast<const float4*>(g + 64 * (kc0 + kc) + 4 * (lane & 15)));
          bb[kc] = __ldg(reinterpret_cast<const float4*>(bta + 64 * (kc0 + kc) + 4 * (lane & 15)));
        }
      wait_counter(word, target);
      float4 xv[KCMAX * 8];
#pragma unroll
      for (int kc = 0; kc < KCMAX; ++kc)
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int row = ww * 16 + it * 2 + (lane >> 4);
          xv[kc * 8 + it] = (kc < nkc && row < M) ? __ldcg(reinterpret_cast<const float4*>(x + (long long)row * d + 64 * (kc0 + kc) + 4 * (lane & 15)))
                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      // row statistics from the groups of 64 features: two threads per row, NC / 2 groups each
      const int srow = wtid >> 1, part = wtid & 1, ngh = NC >> 1;
      float2 st[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        st[i] = (i < ngh && srow < M) ? __ldcg(stats + (long long)srow * NC + part * ngh + i) : make_float2(0.f, 0.f);
      float sm = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) sm += st[i].x;
      sm += __shfl_xor_sync(0xffffffffu, sm, 1);
      const float mean = sm / (float)NC;
      float m2 = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (i < ngh) { const float dv = st[i].x - mean; m2 += st[i].y + 64.0f * dv * dv; }
      m2 += __shfl_xor_sync(0xffffffffu, m2, 1);
      if (part == 0) s_rowstat[srow] = make_float2(mean, rsqrtf(m2 / (float)d + a.eps));
      ff_workers_sync();
#pragma unroll
      for (int kc = 0; kc < KCMAX; ++kc)
        if (kc < nkc) {
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int row = ww * 16 + it * 2 + (lane >> 4);
            const float2 ms = s_rowstat[row];
            const float4 v = xv[kc * 8 + it];
            uint32_t lo = 0u, hi = 0u;
            if (row < M) {
              lo = pack_bf16((v.x - ms.x) * ms.y * gg[kc].x + bb[kc].x, (v.y - ms.x) * ms.y * gg[kc].y + bb[kc].y);
              hi = pack_bf16((v.z - ms.x) * ms.y * gg[kc].z + bb[kc].z, (v.w - ms.x) * ms.y * gg[kc].w + bb[kc].w);
            }
            const uint32_t unit = (uint32_t)((lane & 15) >> 1) ^ (uint32_t)(row & 7);
            const uint32_t ad = xa + (uint32_t)kc * 16384u + (uint32_t)row * 128u + (unit << 4) + (uint32_t)(lane & 1) * 8u;
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(ad), "r"(lo), "r"(hi) : "memory");
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(ad + 8192u), "r"(lo), "r"(hi) : "memory");
            if (y != nullptr && row < M)
              *reinterpret_cast<uint2*>(y + (long long)row * d + 64 * (kc0 + kc) + 4 * (lane & 15)) = make_uint2(lo, hi);
          }
        }
      fence_proxy_async_smem();
      mbar_arrive(bar_xa);
    };
    // Mean and sum of squared deviations of 64 features held four per thread by 16 consecutive lanes.
    auto group_stats = [&](const float4& v, float& mu, float& q) {
      float sm = (v.x + v.y) + (v.z + v.w);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) sm += __shfl_xor_sync(0xffffffffu, sm, o);
      mu = sm * (1.0f / 64.0f);
      const float d0 = v.x - mu, d1 = v.y - mu, d2 = v.z - mu, d3 = v.w - mu;
      q = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    };
    // Residual epilogue of a product whose cluster owns features [64c, 64c+64): item = (token, four features);
    // xres (the item's four values of the residual stream, which this thread also wrote last time) += sum + bias;
    // leaves the (mean, sum of squared deviations) of the 64 features.
    float4 xres[Cfg::kRounds];
#pragma unroll
    for (int rd = 0; rd < Cfg::kRounds; ++rd) xres[rd] = make_float4(0.f, 0.f, 0.f, 0.f);
    auto residual_epilogue = [&](const float* bias, float* xout, float2* stats_out) {
      const int f4 = (wtid & 15) * 4, col = 64 * c + f4;
      const float4 bv = __ldg(reinterpret_cast<const float4*>(bias + col));
      rb_wait();
#pragma unroll
      for (int rd = 0; rd < Cfg::kRounds; ++rd) {
        const int tl = (wtid >> 4) + 8 * rd, m = tok0 + tl;
        const bool mine = tl < ntok;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (mine) {
          const float4 s = rb_sum4(64, tl, f4);
          v = make_float4(xres[rd].x + (s.x + bv.x), xres[rd].y + (s.y + bv.y), xres[rd].z + (s.z + bv.z), xres[rd].w + (s.w + bv.w));
          xres[rd] = v;
          if (m < M) *reinterpret_cast<float4*>(xout + (long long)m * d + col) = v;
        }
        float mu, q;
        group_stats(v, mu, q);
        if (mine && (wtid & 15) == 0 && m < M) stats_out[(long long)m * NC + c] = make_float2(mu, q);
      }
    };

    grid_dep_wait();
    plan();
    // ---------------------------------------------------------------- embedding (tree build + embed)
    {
      const int f4 = (wtid & 15) * 4, col = 64 * c + f4;
#pragma unroll
      for (int rd = 0; rd < Cfg::kRounds; ++rd) {
        const int tl = (wtid >> 4) + 8 * rd, m = tok0 + tl;
        const bool mine = tl < ntok;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (mine && m < M) {
          const int depth = a.tree.depth[m];
          int tok;
          if (a.override_tokens) tok = a.override_tokens[m];
          else if (m == 0) tok = a.root[0];
          else tok = a.topk[(depth - 1) * a.draft_topk + a.tree.rank[m]];
          const bool live = m < nv;
          if (!live) tok = 0;
          int pos = ctx + depth;
          if (pos >= a.max_pos) { if (live && (wtid & 15) == 0) atomicOr(err, kErrCapacity); pos = a.max_pos - 1; }
          const bf16* e;
          if (tok >= 0 && tok < a.vocab) e = a.emb_audio + (long long)tok * d;
          else if (tok >= a.vocab && tok < a.vocab + a.n_phonemes) e = a.emb_phon + (long long)(tok - a.vocab) * d;
          else { if (live && (wtid & 15) == 0) atomicOr(err, kErrCapacity); e = a.emb_audio; }
          const bf16* p = a.pos + (long long)pos * d;
          const uint2 ev = *reinterpret_cast<const uint2*>(e + col), pv = *reinterpret_cast<const uint2*>(p + col);
          const __nv_bfloat162 e0 = *reinterpret_cast<const __nv_bfloat162*>(&ev.x), e1 = *reinterpret_cast<const __nv_bfloat162*>(&ev.y);
          const __nv_bfloat162 q0 = *reinterpret_cast<const __nv_bfloat162*>(&pv.x), q1 = *reinterpret_cast<const __nv_bfloat162*>(&pv.y);
          v.x = __low2float(e0) + __low2float(q0); v.y = __high2float(e0) + __high2float(q0);
          v.z = __low2float(e1) + __low2float(q1); v.w = __high2float(e1) + __high2float(q1);
          *reinterpret_cast<float4*>(a.xa + (long long)m * d + col) = v;
          xres[rd] = v;
          if ((wtid & 15) == 0) {
            long long row = -1;
            if (live) {
              const int slot = ctx + m;
              const long long blk = kv_block_of(a.block_table, a.geom, 0, slot, err);
              if (blk >= 0) row = a.geom.elem(blk, 0, 0, slot % kKvBlock);
            }
            s_kvrow[tl] = row;
            if (c == 0) { a.tokens[m] = tok; a.kv_row[m] = row; }
          }
        } else if (mine && (wtid & 15) == 0) {
          s_kvrow[tl] = -1;
        }
        float mu, q;
        group_stats(v, mu, q);
        if (mine && (wtid & 15) == 0 && m < M) a.stats_a[(long long)m * NC + c] = make_float2(mu, q);
      }
      publish(kFfSyncXa, false);
    }

    const int ntile = np_mine + ((rank == CS - 1 && nv > 0) ? 1 : 0);
    unsigned long long anc_lo = 0ull;
    if (tok_t < nv && tok_t < M) { unsigned long long hi_unused; a.tree.anc_of(0, tok_t, anc_lo, hi_unused); }

    for (int l = 0; l < L; ++l) {
      const long long lb = (long long)l * a.layer_stride;
      auto lvec = [&](const float* p0_) { return reinterpret_cast<const float*>(reinterpret_cast<const char*>(p0_) + lb); };
      bf16* pool_l = a.kv_pool + (long long)l * a.geom.layer_stride;
      // ---------------------------------------------------------------- q/k/v of head c
      build_ln(a.xa, a.stats_a, lvec(a.ln1_g), lvec(a.ln1_b), kFfSyncXa, (uint32_t)(G * (l + 1)), nullptr);
      send_partial(192, true);
      {
        const float* bq = lvec(a.bqkv);
        rb_wait();
        for (int it = wtid; it < ntok * 24; it += kFfWorkers) {
          const int tl = it / 24, u = it % 24, m = tok0 + tl;
          const int part = u >> 3, j0 = (u & 7) * 8;
          const float4 s0 = rb_sum4(192, tl, 8 * u), s1 = rb_sum4(192, tl, 8 * u + 4);
          const float* bp = bq + part * d + c * 64 + j0;
          const float4 b0v = __ldg(reinterpret_cast<const float4*>(bp)), b1v = __ldg(reinterpret_cast<const float4*>(bp + 4));
          const float v8[8] = {s0.x + b0v.x, s0.y + b0v.y, s0.z + b0v.z, s0.w + b0v.w, s1.x + b1v.x, s1.y + b1v.y, s1.z + b1v.z, s1.w + b1v.w};
          const uint4 val = ff_pack8(v8);
          // the row goes to this CTA's own shared memory ([token][q | k | v], 384 bytes), where the peers fetch it;
          // k and v also go to the cache slot of the node
          ff_st_shared_u4(qo + (uint32_t)(tl * 384 + u * 16), val);
          if (m < M && part != 0) {
            const long long row = s_kvrow[tl];
            if (row >= 0) *reinterpret_cast<uint4*>(pool_l + row + (part - 1) * kv_stride + (long long)c * tile_elems + j0) = val;
          }
        }
        ff_fence_cluster();
        __syncwarp();
        if (lane == 0)
          for (uint32_t p = 0; p < (uint32_t)CS; ++p) ff_arrive_remote(ff_mapa(bar_qkv, p));
        rb_done();
        // every owner has staged its rows: fetch the q rows of all tokens into the Q tile (each at r and r + 64) and,
        // in the CTA that scores the tree's own keys, the k and v rows into their tiles
        ff_wait([&] { return ff_try_wait_cluster(bar_qkv, n_qkv & 1); }, err, abort_flag);
        ++n_qkv;
        {
          const int nparts = rank == CS - 1 ? 3 : 1;
          for (int it = wtid; it < nparts * 512; it += kFfWorkers) {
            const int part = it >> 9, m = (it >> 3) & 63, u = it & 7;
            if (m < M) {
              const int ow = ff_owner(m, 64, CS);
              int of, oc;
              ff_split(64, CS, ow, of, oc);
              const uint4 val = ff_ld_cluster_u4(ff_mapa(qo + (uint32_t)((m - of) * 384 + part * 128 + u * 16), (uint32_t)ow));
              const uint32_t off = (uint32_t)m * 128u + ((uint32_t)(u ^ (m & 7)) << 4);
              if (part == 0) { ff_st_shared_u4(xa + off, val); ff_st_shared_u4(xa + 8192u + off, val); }
              else ff_st_shared_u4(xa + (part == 1 ? 16384u : 24576u) + off, val);
            }
          }
          fence_proxy_async_smem();
          mbar_arrive(bar_q);
        }
      }
      // ---------------------------------------------------------------- attention: this CTA's pages
      {
        float m_run = -INFINITY, l_run = 0.f;
        for (int t0 = 0; t0 < ntile; t0 += kFfGroup) {
          const int npg = min(kFfGroup, ntile - t0);
          wait_bar(bar_s, n_s);
          tc_fence_after();
          float mx = -INFINITY;
          bool zeroed = false;
          for (int pi = 0; pi < npg; ++pi) {
            const int t = t0 + pi;
            float sc[32];
            tmem_ld32(trow + kFfColS + 64 * pi + 32 * half_t, sc);
            uint32_t vis;
            if (t < np_mine) {
              const int rem = ctx - ((p0 + t) * kKvBlock + 32 * half_t);
              vis = rem >= 32 ? 0xffffffffu : (rem <= 0 ? 0u : ((1u << rem) - 1u));
              // rows of the V tile past the context may hold anything: zero them (their weights are zero)
              const int valid = ctx - (p0 + t) * kKvBlock;
              if (valid < kKvBlock) {
                if (wtid < kKvBlock && wtid >= valid) {
                  const int seq = l * ipl + offKV + t;
                  uint4* vr = reinterpret_cast<uint4*>(ring_p + (seq % R) * kFfSlotBytes + kFfTileBytes + wtid * 128);
#pragma unroll
                  for (int q8 = 0; q8 < 8; ++q8) vr[q8] = make_uint4(0, 0, 0, 0);
                }
                zeroed = true;
              }
            } else {
              vis = (uint32_t)(anc_lo >> (32 * half_t));
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) mx = fmaxf(mx, ((vis >> j) & 1u) ? sc[j] : -INFINITY);
          }
          mx *= a.scale_log2e;
          const float m_new = fmaxf(m_run, mx);
          if (t0 > 0) {
            // bring the accumulator to the new maximum once the previous group's P V has completed
            wait_bar(bar_o, n_o);
            tc_fence_after();
            const float factor = (m_run == -INFINITY) ? 0.f : fast_exp2(m_run - m_new);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              float ot[32];
              tmem_ld32(trow + kFfColO + 32 * hh, ot);
              uint32_t ob[32];
#pragma unroll
              for (int e = 0; e < 32; ++e) ob[e] = __float_as_uint(ot[e] * factor);
              tmem_st32(trow + kFfColO + 32 * hh, ob);
            }
            l_run *= factor;
          }
          m_run = m_new;
          const float m_sub = (m_new == -INFINITY) ? 0.f : m_new;
          for (int pi = 0; pi < npg; ++pi) {
            const int t = t0 + pi;
            float sc[32];
            const uint32_t tsp = trow + kFfColS + 64 * pi;
            tmem_ld32(tsp + 32 * half_t, sc);
            uint32_t vis;
            if (t < np_mine) {
              const int rem = ctx - ((p0 + t) * kKvBlock + 32 * half_t);
              vis = rem >= 32 ? 0xffffffffu : (rem <= 0 ? 0u : ((1u << rem) - 1u));
            } else {
              vis = (uint32_t)(anc_lo >> (32 * half_t));
            }
            float psum = 0.f;
            uint32_t hv[16], lv[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float sa = ((vis >> (2 * j)) & 1u) ? sc[2 * j] : -INFINITY;
              const float sb = ((vis >> (2 * j + 1)) & 1u) ? sc[2 * j + 1] : -INFINITY;
              const float pa = fast_exp2(fmaf(sa, a.scale_log2e, -m_sub));
              const float pb = fast_exp2(fmaf(sb, a.scale_log2e, -m_sub));
              psum += pa + pb;
              hv[j] = pack_bf16(pa, pb);
              const float ha = __uint_as_float(hv[j] << 16), hb = __uint_as_float(hv[j] & 0xffff0000u);
              lv[j] = pack_bf16(pa - ha, pb - hb);
            }
            l_run += psum;
            uint32_t zero[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) zero[j] = 0u;
            tmem_st16(tsp + 16 * half_t, hv);
            tmem_st16(tsp + 16 * (1 - half_t), zero);
            tmem_st16(tsp + 32 + 16 * half_t, lv);
            tmem_st16(tsp + 32 + 16 * (1 - half_t), zero);
          }
          tmem_st_wait();
          tc_fence_before();
          if (zeroed) fence_proxy_async_smem();
          mbar_arrive(bar_p);
        }
        // this lane's partial: 64 output features, the sum of weights and their scaling maximum -> the token's owner
        float oacc[64];
        if (ntile > 0) {
          wait_bar(bar_o, n_o);
          tc_fence_after();
          tmem_ld32(trow + kFfColO, oacc);
          tmem_ld32(trow + kFfColO + 32, oacc + 32);
        } else {
#pragma unroll
          for (int e = 0; e < 64; ++e) oacc[e] = 0.f;
        }
        rb_begin();
        {
          const uint32_t dst = rb + (uint32_t)(lane_t * 68) * 4u;      // [lane = copy * 64 + token][64 features, l, m, pad]
#pragma unroll
          for (int i = 0; i < 16; ++i) ff_st_shared_f4(dst + 16u * i, oacc[4 * i], oacc[4 * i + 1], oacc[4 * i + 2], oacc[4 * i + 3]);
          ff_st_shared_f4(dst + 256u, l_run, m_run, 0.f, 0.f);
        }
        rb_sent();
        tc_fence_before();
        // owner: merge the 2 CS partials of each of its tokens
        rb_wait();
        {
          const int f4 = (wtid & 15) * 4;
#pragma unroll
          for (int rd = 0; rd < Cfg::kRounds; ++rd) {
            const int tl = (wtid >> 4) + 8 * rd, m = tok0 + tl;
            if (tl < ntok) {
              float mm[2 * CS], ll[2 * CS];
              float4 ovv[2 * CS];
              float mxx = -INFINITY;
#pragma unroll
              for (int p = 0; p < 2 * CS; ++p) {            // partial p: CTA p / 2, copy p % 2 of the token
                const uint32_t src = ff_mapa(rb + (uint32_t)(((p & 1) * 64 + m) * 68) * 4u, (uint32_t)(p >> 1));
                const float4 lm = ff_ld_cluster_f4(src + 256u);
                ovv[p] = ff_ld_cluster_f4(src + (uint32_t)f4 * 4u);
                ll[p] = lm.x; mm[p] = lm.y;
              }
#pragma unroll
              for (int p = 0; p < 2 * CS; ++p) mxx = fmaxf(mxx, mm[p]);
              float Ls = 0.f;
              float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int p = 0; p < 2 * CS; ++p) {
                const float w = (mm[p] == -INFINITY) ? 0.f : exp2f(mm[p] - mxx);
                const float4 ov = ovv[p];
                Ls = fmaf(ll[p], w, Ls);
                o4.x = fmaf(ov.x, w, o4.x); o4.y = fmaf(ov.y, w, o4.y); o4.z = fmaf(ov.z, w, o4.z); o4.w = fmaf(ov.w, w, o4.w);
              }
              if (m < M) {
                const float inv = (m < nv && Ls > 0.f) ? 1.f / Ls : 0.f;
                uint2 v;
                v.x = pack_bf16(o4.x * inv, o4.y * inv);
                v.y = pack_bf16(o4.z * inv, o4.w * inv);
                *reinterpret_cast<uint2*>(a.o + (long long)m * d + c * 64 + f4) = v;
                if (a.attn_tap) *reinterpret_cast<uint2*>(a.attn_tap + ((long long)l * M + m) * d + c * 64 + f4) = v;
              }
            }
          }
        }
        publish(kFfSyncO + c, true);
        rb_done();
      }
      // ---------------------------------------------------------------- output projection, rows [64c, 64c+64)
      send_partial(64, false);
      residual_epilogue(lvec(a.bo), a.xb, a.stats_b);
      publish(kFfSyncXb, false);
      rb_done();
      // ---------------------------------------------------------------- first feed-forward matrix, rows [c n1, (c+1) n1)
      build_ln(a.xb, a.stats_b, lvec(a.ln2_g), lvec(a.ln2_b), kFfSyncXb, (uint32_t)(G * (l + 1)), nullptr);
      send_partial(n1, true);
      {
        const float* b1 = lvec(a.b1);
        const int units = n1 / 8;                            // 16-byte units per token
        rb_wait();
        for (int it = wtid; it < ntok * units; it += kFfWorkers) {
          const int tl = it / units, u = it % units, m = tok0 + tl;
          const float4 s0 = rb_sum4(n1, tl, 8 * u), s1 = rb_sum4(n1, tl, 8 * u + 4);
          const float* bp = b1 + c * n1 + 8 * u;
          const float4 b0v = __ldg(reinterpret_cast<const float4*>(bp)), b1v = __ldg(reinterpret_cast<const float4*>(bp + 4));
          const float v8[8] = {fmaxf(s0.x + b0v.x, 0.f), fmaxf(s0.y + b0v.y, 0.f), fmaxf(s0.z + b0v.z, 0.f), fmaxf(s0.w + b0v.w, 0.f),
                               fmaxf(s1.x + b1v.x, 0.f), fmaxf(s1.y + b1v.y, 0.f), fmaxf(s1.z + b1v.z, 0.f), fmaxf(s1.w + b1v.w, 0.f)};
          if (m < M) *reinterpret_cast<uint4*>(a.mid + (long long)m * F + c * n1 + 8 * u) = ff_pack8(v8);
        }
        publish(kFfSyncMid + c, true);
        rb_done();
      }
      // ---------------------------------------------------------------- second feed-forward matrix, rows [64c, 64c+64)
      send_partial(64, false);
      residual_epilogue(lvec(a.b2), a.xa, a.stats_a);
      publish(kFfSyncXa, false);
      rb_done();
    }
    // ---------------------------------------------------------------- final LayerNorm + vocabulary head
    if (lm_mine) {
      bool first = true;
      for (int t = c; t < nlm; t += NC) {
        if (first) {
          build_ln(a.xa, a.stats_a, a.lnf_g, a.lnf_b, kFfSyncXa, (uint32_t)(G * (L + 1)), c == 0 ? a.hfinal : nullptr);
          first = false;
        }
        send_partial(128, true);
        rb_wait();
        for (int it = wtid; it < ntok * 32; it += kFfWorkers) {
          const int tl = it >> 5, f4 = (it & 31) * 4, m = tok0 + tl;
          const float4 s = rb_sum4(128, tl, f4);
          if (m < M) *reinterpret_cast<float4*>(a.logits + (long long)m * a.vpad + 128 * t + f4) = s;
        }
        rb_done();
      }
    }
  }

  // ---- common exit: nothing of this CTA may be in flight, and no peer may still address its shared memory
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && tid == 0) {
    // loads of this CTA that were still in flight when a wait ran out: give them time to land
    const unsigned long long t0 = ff_timer();
    while (ff_timer() - t0 < 200000ull) {}
  }
  cluster_sync_all();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem, 512);
  // the last CTA to finish clears the counters for the next pass
  if (tid == 0) {
    __threadfence();
    const uint32_t prev = atomicAdd(a.sync + kFfSyncDone, 1u);
    if (prev == (uint32_t)G - 1u) {
      for (int i = 0; i < kFfSyncWords; ++i) a.sync[i] = 0u;
      __threadfence();
    }
  }
}

}  // namespace vadusa
