// libvadusa: host engine and C ABI.  Every step of the draft-and-verify path runs in
// the kernels included below; this file only validates, lays out memory and launches.
#include <cuda_runtime.h>
#include <stdarg.h>

#include <type_traits>

#include <algorithm>
#include <map>
#include <new>
#include <string>
#include <tuple>

#include "accept.cuh"
#include "attention_simt.cuh"
#include "attention_tc.cuh"
#include "attention_prefill_tc.cuh"
#include "attention_stream_tc.cuh"
#include "elementwise.cuh"
#include "fit.cuh"
#include "fwd_fused.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "layout.h"
#include "select.cuh"

using namespace vadusa;

struct LayerW {
  const float *ln1_g, *ln1_b, *bqkv, *bo, *ln2_g, *ln2_b, *b1, *b2;
  const void *wqkv, *wo, *w1, *w2;
};

struct vadusa_ctx {
  vadusa_config cfg;
  std::vector<LayerW> layers;
  const void *emb_audio = nullptr, *emb_phon = nullptr, *pos = nullptr, *lm = nullptr, *dw = nullptr, *du = nullptr;
  const float *lnf_g = nullptr, *lnf_b = nullptr, *db = nullptr;
  long long dw_stride = 0, du_stride = 0;     // bytes between draft heads
  WorkspaceLayout ws;
  std::vector<TensorDesc> wl;
  const char* blob = nullptr;
  char* wsp = nullptr;
  cudaStream_t stream = nullptr;
  int batch = 0;
  const float* logit_bias = nullptr;   // caller's [batch][logit_bias_ld] fp32 added to the base head's logits (sampler hook)
  int logit_bias_ld = 0;
  int n_nodes = 0;            // current tree size (0: none set)
  int tree_per_seq = 0;
  int max_rank_used = 0;
  int tree_max_depth = 0;
  // draft-head fitting (vadusa_fit_*): the caller's state buffer and the schedule
  char* fit = nullptr;
  int fit_tokens = 0, fit_step = 0, fit_warmup = 0;
  float fit_lambda = 0.f, fit_lr = 0.f;
  void* pf_tap = nullptr;     // where prefill also leaves the final hidden state of every prefix token ([batch][stride][d])
  int pf_tap_stride = 0;
  int pf_tiles = 0;           // > 0 while a prefill pass runs: attention CTAs of the pass (pairs of chunks), listed in ws.pf_pairs
  int att_stream = 0;         // batches: attention as one persistent kernel over the stream of K/V pages (0: one CTA per head and sequence)
  int fused_enabled = 0;      // single-sequence passes run as one persistent kernel (0: no, 1: yes, 6 / 8: with that cluster size)
  int fused_clusters = -1;    // clusters of that kernel that can be resident at once on this device (-1: not asked yet)
  int fused_cs = -1;          // CTAs per cluster chosen for it (8 or 6; 0: the device cannot hold one cluster per head)
  int fused_n8 = 0, fused_n6 = 0;
  long long ctx_bound = 0;    // host-side upper bound of the longest context (grows by the longest path per commit)
  long long ctx_lo = 0;       // host-side lower estimate of it (one token per iteration); exact after begin, prefill, get_lengths
  const int32_t* block_table = nullptr;
  bool have_draft = false, have_verify = false;
  int64_t launches = 0;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr, ev_poll = nullptr;
  int32_t* h_pinned = nullptr;     // [2]: done_count, err
  char err[512] = {0};
  // TMA descriptors of the operands of the tensor-core products, made on first use
  typedef std::tuple<const void*, int, int, int, int, long long> MapKey;   // ptr, rows, K, box rows, batches, batch stride
  std::map<MapKey, CUtensorMap> maps;
  void* encode_fn = nullptr;       // cuTensorMapEncodeTiled, resolved through the runtime
  // CUDA graphs of the launch sequences of the hot calls, keyed by their baked-in arguments
  struct GraphRec { cudaGraphExec_t exec = nullptr; int seen = 0; int64_t launches = 0; };
  std::map<std::string, GraphRec> graphs;
  // per-kernel timing (vadusa_profile_begin/end): one event pair per launch
  struct ProfRec { cudaEvent_t a, b; int cls; };
  bool prof_on = false, prof_pending = false;
  std::vector<ProfRec> prof;
};

enum KClass { K_EMBED, K_LAYERNORM, K_GEMM_QKV, K_ATTENTION, K_GEMM_OUT, K_GEMM_FFN1, K_GEMM_FFN2, K_GEMM_LM,
              K_DRAFT_HIDDEN, K_DRAFT_LOGITS, K_DRAFT_SELECT, K_ACCEPT, K_COMMIT, K_MISC, K_FUSED, K_NCLASS };
static const char* const kClassName[K_NCLASS] = {
    "tree_embed", "layernorm", "gemm_qkv", "tree_attention", "gemm_out", "gemm_ffn1", "gemm_ffn2", "gemm_lm",
    "draft_hidden", "draft_logits", "draft_select", "accept", "commit", "misc", "fused_forward"};

namespace {

vadusa_status fail(vadusa_ctx* c, vadusa_status s, const char* fmt, ...) {
  if (c) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c->err, sizeof(c->err), fmt, ap);
    va_end(ap);
  }
  return s;
}

#define CU(call)                                                                                   \
  do {                                                                                             \
    cudaError_t e_ = (call);                                                                       \
    if (e_ != cudaSuccess) return fail(ctx, VADUSA_ECUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

#define LAUNCH_CHECK()                                                                             \
  do {                                                                                             \
    cudaError_t e_ = cudaGetLastError();                                                           \
    if (e_ != cudaSuccess) return fail(ctx, VADUSA_ECUDA, "kernel launch: %s", cudaGetErrorString(e_)); \
    ctx->launches++;                                                                               \
    if (ctx->prof_pending) { cudaEventRecord(ctx->prof.back().b, ctx->stream); ctx->prof_pending = false; } \
  } while (0)

// Call right before a kernel launch: when profiling is on, brackets the launch with events.
void PROF(vadusa_ctx* c, int cls) {
  if (!c->prof_on) return;
  vadusa_ctx::ProfRec r;
  r.cls = cls;
  if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
  cudaEventRecord(r.a, c->stream);
  c->prof.push_back(r);
  c->prof_pending = true;
}

template <typename P> P* wsptr(vadusa_ctx* c, int64_t off) { return reinterpret_cast<P*>(c->wsp + off); }

const TensorDesc* find(const vadusa_ctx* c, const std::string& name) {
  for (const auto& t : c->wl)
    if (t.name == name) return &t;
  return nullptr;
}
const void* wraw(const vadusa_ctx* c, const std::string& name) {
  const TensorDesc* t = find(c, name);
  return t ? c->blob + t->offset : nullptr;
}

void resolve_weights(vadusa_ctx* c) {
  auto f = [&](const std::string& n) { return reinterpret_cast<const float*>(wraw(c, n)); };
  c->layers.resize(c->cfg.n_layers);
  for (int l = 0; l < c->cfg.n_layers; ++l) {
    const std::string p = "l" + std::to_string(l) + ".";
    LayerW& w = c->layers[l];
    w.ln1_g = f(p + "ln1_g"); w.ln1_b = f(p + "ln1_b"); w.bqkv = f(p + "bqkv"); w.bo = f(p + "bo");
    w.ln2_g = f(p + "ln2_g"); w.ln2_b = f(p + "ln2_b"); w.b1 = f(p + "b1"); w.b2 = f(p + "b2");
    w.wqkv = wraw(c, p + "wqkv"); w.wo = wraw(c, p + "wo"); w.w1 = wraw(c, p + "w1"); w.w2 = wraw(c, p + "w2");
  }
  c->emb_audio = wraw(c, "emb_audio"); c->emb_phon = wraw(c, "emb_phon"); c->pos = wraw(c, "pos");
  c->lnf_g = f("lnf_g"); c->lnf_b = f("lnf_b"); c->lm = wraw(c, "lm");
  c->dw = wraw(c, "draft0.w"); c->db = f("draft0.b"); c->du = wraw(c, "draft0.u");
  if (c->cfg.n_draft_heads > 1) {
    c->dw_stride = find(c, "draft1.w")->offset - find(c, "draft0.w")->offset;
    c->du_stride = find(c, "draft1.u")->offset - find(c, "draft0.u")->offset;
  }
}
template <typename T> const T* as(const void* p) { return reinterpret_cast<const T*>(p); }

uint32_t* err_word(vadusa_ctx* c) { return wsptr<uint32_t>(c, c->ws.scalars); }
int32_t* done_word(vadusa_ctx* c) { return wsptr<int32_t>(c, c->ws.scalars) + 1; }

KvGeom geom_of(const vadusa_ctx* c) {
  KvGeom g;
  g.n_heads = c->cfg.n_heads;
  g.head_dim = c->cfg.d_model / c->cfg.n_heads;
  g.max_blocks_per_seq = c->cfg.max_blocks_per_seq;
  g.num_blocks = c->cfg.kv_num_blocks;
  g.layer_stride = (long long)c->cfg.kv_num_blocks * 2 * c->cfg.d_model * kKvBlock;
  return g;
}

TreeView tree_of(vadusa_ctx* c, bool chain) {
  TreeView t;
  if (chain) {
    t.parent = wsptr<int32_t>(c, c->ws.chain_parent);
    t.depth = wsptr<int32_t>(c, c->ws.chain_depth);
    t.rank = wsptr<int32_t>(c, c->ws.chain_rank);
    t.anc = wsptr<unsigned long long>(c, c->ws.chain_anc);
    t.n_nodes = c->cfg.max_tree_nodes;
    t.per_seq = 0;
  } else {
    t.parent = wsptr<int32_t>(c, c->ws.tree_parent);
    t.depth = wsptr<int32_t>(c, c->ws.tree_depth);
    t.rank = wsptr<int32_t>(c, c->ws.tree_rank);
    t.anc = wsptr<unsigned long long>(c, c->ws.tree_anc);
    t.n_nodes = c->n_nodes;
    t.per_seq = c->tree_per_seq;
  }
  return t;
}

SeqState state_of(vadusa_ctx* c, int32_t* out_tokens, int out_cap, int target) {
  SeqState s;
  s.ctx_len = wsptr<int32_t>(c, c->ws.ctx_len);
  s.nvalid = wsptr<int32_t>(c, c->ws.nvalid);
  s.gen_count = wsptr<int32_t>(c, c->ws.gen_count);
  s.commit_base = wsptr<int32_t>(c, c->ws.commit_base);
  s.commit_len = wsptr<int32_t>(c, c->ws.commit_len);
  s.commit_path = wsptr<int32_t>(c, c->ws.commit_path);
  s.best = wsptr<int32_t>(c, c->ws.best);
  s.out_tokens = out_tokens;
  s.done_count = done_word(c);
  s.out_cap = out_cap;
  s.target = target;
  s.stats = wsptr<unsigned long long>(c, c->ws.acc_stats);
  return s;
}
static_assert(kStatDepth == VADUSA_MAX_DEPTH && kStatTopk == VADUSA_MAX_DRAFT_TOPK, "statistics table follows the C ABI's maxima");

vadusa_status sampling_dev(vadusa_ctx* ctx, const vadusa_sampling* s, SamplingDev* o) {
  if (!s) return fail(ctx, VADUSA_EINVAL, "sampling is NULL");
  if (s->tau < 1) return fail(ctx, VADUSA_EINVAL, "tau must be >= 1");
  if (!(s->temperature >= 0.f)) return fail(ctx, VADUSA_EINVAL, "temperature must be >= 0");
  if (!(s->top_p > 0.f)) return fail(ctx, VADUSA_EINVAL, "top_p must be > 0");
  if (s->accept_rule != 0 && s->accept_rule != 1) return fail(ctx, VADUSA_EINVAL, "accept_rule must be 0 or 1");
  memset(o, 0, sizeof(*o));            // the bytes of this struct key the graph cache: no stray padding
  o->tau = s->tau;
  o->temperature = s->temperature;
  o->inv_temperature = s->temperature > 0.f ? (float)(1.0 / (double)s->temperature) : 1.f;
  o->top_p = s->top_p;
  o->eos_masked = s->eos_masked ? 1 : 0;
  o->accept_rule = s->accept_rule;
  o->eos_id = ctx->cfg.vocab - 1;
  o->seed = s->seed;
  o->bias = ctx->logit_bias;
  o->bias_ld = ctx->logit_bias_ld;
  return VADUSA_OK;
}

// ---- typed engine ------------------------------------------------------------------

template <typename T, typename Epi>
vadusa_status gemm(vadusa_ctx* ctx, int cls, const T* A, const T* W, int M, int N, int K, int batches, long long a_z,
                   long long w_z, const Epi& epi) {
  dim3 grid((N + 63) / 64, (M + 63) / 64, batches);
  PROF(ctx, cls);
  gemm_simt_kernel<T, Epi><<<grid, 256, 0, ctx->stream>>>(A, W, M, N, K, a_z, w_z, epi);
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// ---- tensor-core products (bf16 models) ------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Descriptor of a row-major bf16 matrix [batches][rows][K] read in boxes of box_rows x 64
// elements with the 128-byte swizzle; rows outside the matrix read as zero.
vadusa_status tensor_map(vadusa_ctx* ctx, const void* ptr, int rows, int K, int box_rows, int batches,
                         long long batch_stride_elems, const CUtensorMap** out) {
  vadusa_ctx::MapKey key(ptr, rows, K, box_rows, batches, batch_stride_elems);
  auto it = ctx->maps.find(key);
  if (it == ctx->maps.end()) {
    if (!ctx->encode_fn) return fail(ctx, VADUSA_ECUDA, "cuTensorMapEncodeTiled is not available");
    CUtensorMap m;
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)batches};
    cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)(batches > 1 ? batch_stride_elems : (long long)rows * K) * 2};
    cuuint32_t box[3] = {(cuuint32_t)kGemmBK, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_fn)(
        &m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, VADUSA_ECUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    it = ctx->maps.emplace(key, m).first;
  }
  *out = &it->second;
  return VADUSA_OK;
}

// X == nullptr with ln != nullptr: the LayerNorm-fused variant (the operand is made in the kernel).
template <int TN, typename Epi, bool LN = false>
vadusa_status launch_gemm_tc(vadusa_ctx* ctx, int cls, const void* X, const void* W, int w_rows, int M, int N, int K,
                             int batches, long long x_z, long long w_z, int ksplit, const Epi& epi,
                             const LnFuse* ln = nullptr) {
  using Cfg = GemmTcCfg<TN>;
  static unsigned long long attr_done = 0ull;              // per device: function attributes belong to a device's context
  const unsigned long long dev_bit = 1ull << (ctx->cfg.device & 63);
  if (!(attr_done & dev_bit)) {
    CU(cudaFuncSetAttribute(gemm_tc_kernel<TN, Epi, LN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemMax));
    CU(cudaFuncSetAttribute(gemm_tc_kernel<TN, Epi, LN>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    CU(cudaFuncSetAttribute(gemm_tc_kernel<TN, Epi, LN>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    attr_done |= dev_bit;
  }
  const int chunks = K / kGemmBK / ksplit;
  const int smem = Cfg::smem_for(chunks, ksplit);
  const CUtensorMap *mw, *mx;
  if (vadusa_status s = tensor_map(ctx, W, w_rows, K, kGemmRowsW, batches, w_z, &mw)) return s;
  if (LN) mx = mw;                                       // unused by the kernel
  else if (vadusa_status s = tensor_map(ctx, X, M, K, TN, batches, x_z, &mx)) return s;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((N + kGemmRowsW - 1) / kGemmRowsW, (M + TN - 1) / TN, batches * ksplit);
  lc.blockDim = dim3(128);
  lc.dynamicSmemBytes = smem;
  lc.stream = ctx->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = ksplit;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel calls griddepcontrol.wait
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = 2;
  PROF(ctx, cls);
  CU(cudaLaunchKernelEx(&lc, gemm_tc_kernel<TN, Epi, LN>, *mw, *mx, M, N, chunks, ksplit, Cfg::stages_for(chunks),
                        Cfg::ring_for(chunks, ksplit), epi, wsptr<float>(ctx, ctx->ws.gemm_part), err_word(ctx),
                        ln ? *ln : LnFuse{}));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// Many-token product on CTA pairs (256 features x TN tokens per pair, no K split).
template <int TN, int ST, typename Epi>
vadusa_status launch_gemm_tc2(vadusa_ctx* ctx, int cls, const void* X, const void* W, int w_rows, int M, int N, int K,
                              const Epi& epi) {
  using Cfg = GemmTc2Cfg<TN, ST>;
  static unsigned long long attr_done = 0ull;              // per device, like launch_gemm_tc
  const unsigned long long dev_bit = 1ull << (ctx->cfg.device & 63);
  if (!(attr_done & dev_bit)) {
    CU(cudaFuncSetAttribute(gemm_tc2_kernel<TN, ST, Epi>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem));
    CU(cudaFuncSetAttribute(gemm_tc2_kernel<TN, ST, Epi>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    attr_done |= dev_bit;
  }
  const CUtensorMap *mw, *mx;
  if (vadusa_status s = tensor_map(ctx, W, w_rows, K, kGemmRowsW, 1, 0, &mw)) return s;
  if (vadusa_status s = tensor_map(ctx, X, M, K, TN / 2, 1, 0, &mx)) return s;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(N / kGemmRowsW, (M + TN - 1) / TN, 1);           // N is a multiple of 256: whole pairs
  lc.blockDim = dim3(128);
  lc.dynamicSmemBytes = Cfg::kSmem;
  lc.stream = ctx->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel calls griddepcontrol.wait
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = 2;
  PROF(ctx, cls);
  CU(cudaLaunchKernelEx(&lc, gemm_tc2_kernel<TN, ST, Epi>, *mw, *mx, M, N, K / kGemmBK, epi, err_word(ctx)));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// Persistent CTA pairs: tiles of 256 features x 256 tokens dealt round-robin to as many pairs as balance the rounds.
template <typename Epi>
vadusa_status launch_gemm_tc2p(vadusa_ctx* ctx, int cls, const void* X, const void* W, int w_rows, int M, int N, int K,
                               const Epi& epi) {
  static unsigned long long attr_done = 0ull;
  const unsigned long long dev_bit = 1ull << (ctx->cfg.device & 63);
  if (!(attr_done & dev_bit)) {
    CU(cudaFuncSetAttribute(gemm_tc2p_kernel<Epi>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmP2Smem));
    CU(cudaFuncSetAttribute(gemm_tc2p_kernel<Epi>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    attr_done |= dev_bit;
  }
  const CUtensorMap *mw, *mx;
  if (vadusa_status s = tensor_map(ctx, W, w_rows, K, kGemmRowsW, 1, 0, &mw)) return s;
  if (vadusa_status s = tensor_map(ctx, X, M, K, kGemmP2TN / 2, 1, 0, &mx)) return s;
  const int tiles = (N / (2 * kGemmRowsW)) * ((M + kGemmP2TN - 1) / kGemmP2TN);
  const int rounds = (tiles + 73) / 74, npairs = (tiles + rounds - 1) / rounds;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(2 * npairs, 1, 1);
  lc.blockDim = dim3(kGemmP2Threads);
  lc.dynamicSmemBytes = kGemmP2Smem;
  lc.stream = ctx->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = 2;
  PROF(ctx, cls);
  CU(cudaLaunchKernelEx(&lc, gemm_tc2p_kernel<Epi>, *mw, *mx, M, N, K / kGemmBK, tiles, epi, err_word(ctx)));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// K split of a product with `tiles` output tiles of tn tokens: about one CTA per SM streams weights.
static int gemm_ksplit(int tiles, int chunks, int tn) {
  int ksplit = 1;
  while (ksplit < kGemmMaxSplit && tiles * ksplit < 148 && chunks % (ksplit * 2) == 0 && ksplit * 2 <= tn &&
         (long long)tiles * ksplit * 2 * tn * kGemmRowsW * 4 <= kGemmPartBytes)
    ksplit *= 2;
  return ksplit;
}

// Does a residual product of N = d_model features over K inputs leave LayerNorm statistics for M
// tokens?  (Its split-K epilogue does; the fused consumer handles at most 64 tokens and 8 groups.)
static bool residual_leaves_stats(int M, int d, int K) {
  if (M > 64 || d % 128 || d / 128 > 8 || K % kGemmBK) return false;
  const int tn = M <= 16 ? 16 : M <= 32 ? 32 : 64;
  return gemm_ksplit(d / kGemmRowsW, K / kGemmBK, tn) >= 2;
}

// LayerNorm(x) * W^T with the normalisation done inside the product kernel from the statistics the
// producer of x left; applies when the tokens fit one tile of at most 64 and the K slices of the
// cluster are 128 columns.  Returns false (nothing launched) when the shape does not qualify.
template <typename Epi>
bool gemm_tc_ln(vadusa_ctx* ctx, int cls, const float* x, const float* g, const float* b, const void* W, int w_rows,
                int M, int N, int K, const Epi& epi, vadusa_status* st, bf16* y = nullptr) {
  if (M > 64 || K % 128 || K / 128 > 8) return false;
  const int tn = M <= 16 ? 16 : M <= 32 ? 32 : 64;
  const int tiles = (N + kGemmRowsW - 1) / kGemmRowsW;
  const int ksplit = K / 128;                            // one CTA of the cluster per group of 128 columns
  if (ksplit < 2 || ksplit > tn || (long long)tiles * ksplit * tn * kGemmRowsW * 4 > kGemmPartBytes) return false;
  const LnFuse ln{x, g, b, wsptr<float2>(ctx, ctx->ws.ln_stats), y, K, ctx->cfg.ln_eps};
  switch (tn) {
    case 16: *st = launch_gemm_tc<16, Epi, true>(ctx, cls, nullptr, W, w_rows, M, N, K, 1, 0, 0, ksplit, epi, &ln); break;
    case 32: *st = launch_gemm_tc<32, Epi, true>(ctx, cls, nullptr, W, w_rows, M, N, K, 1, 0, 0, ksplit, epi, &ln); break;
    default: *st = launch_gemm_tc<64, Epi, true>(ctx, cls, nullptr, W, w_rows, M, N, K, 1, 0, 0, ksplit, epi, &ln); break;
  }
  return true;
}

// Tile width by token count; K split so that about one CTA per SM streams weights.
template <typename Epi>
vadusa_status gemm_tc(vadusa_ctx* ctx, int cls, const void* X, const void* W, int w_rows, int M, int N, int K,
                      int batches, long long x_z, long long w_z, const Epi& epi) {
  // token tile: as narrow as the token count allows for weight streaming; 256 for the tensor-bound shapes
  // when that still gives every SM a CTA pair, else 128
  const int ntiles_n = (N + kGemmRowsW - 1) / kGemmRowsW;
  // tensor-bound shapes whose features come in whole pairs of tiles: CTA pairs, when they fill the SMs.  Of
  // the 256-token tile (two CTAs per SM) and the 128-token tile (two per SM with four stages when all CTAs are
  // resident at once, else three per SM with three stages) the one whose last wave is fuller; ties to the wider.
  if (M > 512 && batches == 1 && N % (2 * kGemmRowsW) == 0) {
    // at least two full rounds of 256 x 256 tiles per pair: resident pairs whose epilogue runs under the next tile
    if ((N / (2 * kGemmRowsW)) * ((M + 255) / 256) >= 148) return launch_gemm_tc2p(ctx, cls, X, W, w_rows, M, N, K, epi);
    auto fill = [](int ctas, int slots) { return (double)ctas / (double)(((ctas + slots - 1) / slots) * slots); };
    const int c256 = ntiles_n * ((M + 255) / 256), c128 = ntiles_n * ((M + 127) / 128);
    const double f256 = c256 >= 128 ? fill(c256, 296) : 0.0;
    const double f128 = c128 >= 128 ? fill(c128, c128 <= 296 ? 296 : 444) : 0.0;
    if (f256 > 0.0 && f256 >= f128) return launch_gemm_tc2<256, 3>(ctx, cls, X, W, w_rows, M, N, K, epi);
    if (f128 > 0.0 && c128 <= 296) return launch_gemm_tc2<128, 4>(ctx, cls, X, W, w_rows, M, N, K, epi);
    if (f128 > 0.0) return launch_gemm_tc2<128, 3>(ctx, cls, X, W, w_rows, M, N, K, epi);
  }
  int tn = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : M <= 1024 ? 128 : 256;
  if (tn == 256 && ntiles_n * ((M + 255) / 256) * batches < 200) tn = 128;
  const int tiles = ((N + kGemmRowsW - 1) / kGemmRowsW) * ((M + tn - 1) / tn) * batches;
  const int ksplit = gemm_ksplit(tiles, K / kGemmBK, tn);
  switch (tn) {
    case 16: return launch_gemm_tc<16>(ctx, cls, X, W, w_rows, M, N, K, batches, x_z, w_z, ksplit, epi);
    case 32: return launch_gemm_tc<32>(ctx, cls, X, W, w_rows, M, N, K, batches, x_z, w_z, ksplit, epi);
    case 64: return launch_gemm_tc<64>(ctx, cls, X, W, w_rows, M, N, K, batches, x_z, w_z, ksplit, epi);
    case 128: return launch_gemm_tc<128>(ctx, cls, X, W, w_rows, M, N, K, batches, x_z, w_z, ksplit, epi);
    default: return launch_gemm_tc<256>(ctx, cls, X, W, w_rows, M, N, K, batches, x_z, w_z, ksplit, epi);
  }
}

// Product dispatch by model type: fp32 models use plain FMA arithmetic, bf16 models the
// tensor cores (K must be a multiple of 64 there, else the FMA kernel serves).
template <typename T, typename Epi>
vadusa_status product(vadusa_ctx* ctx, int cls, const T* X, const T* W, int w_rows, int M, int N, int K, int batches,
                      long long x_z, long long w_z, const Epi& epi) {
  if constexpr (std::is_same<T, bf16>::value) {
    if (K % kGemmBK == 0) return gemm_tc(ctx, cls, X, W, w_rows, M, N, K, batches, x_z, w_z, epi);
  }
  return gemm<T>(ctx, cls, X, W, M, N, K, batches, x_z, w_z, epi);
}

// LayerNorm followed by a product, in one kernel where the shape allows (bf16 models, few tokens).
template <typename T, typename Epi>
bool ln_product(vadusa_ctx* ctx, int cls, const float* x, const float* g, const float* b, const T* W, int w_rows, int M,
                int N, int K, const Epi& epi, vadusa_status* st, T* y = nullptr) {
  if constexpr (std::is_same<T, bf16>::value) return gemm_tc_ln(ctx, cls, x, g, b, W, w_rows, M, N, K, epi, st, y);
  return false;
}

// KV splits of the tensor-core attention: enough CTAs for about two per SM even at batch 1, but no more than four
// per (head, sequence) while the contexts are short (a 16-head pass over 400-1100 tokens: 64 CTAs of two to five
// pages leave SMs to the next kernel's early CTAs and their weight loads, 128 CTAs of one or two pages do not;
// 0.538 -> 0.528 ms per step).  The estimate of the context is the host's lower one: never behind by more than
// the tokens accepted beyond one per iteration since the last exact value.
// (Ragged batches are balanced by visiting the sequences longest first, see seq_order_kernel.)
constexpr long long kAttLongContext = 1536;
int attention_splits(const vadusa_ctx* ctx, int n_nodes) {
  int splits = 1;
  const int ntile = (n_nodes + 63) / 64;                 // CTAs per (head, sequence): one per 64 nodes
  const int cap = ctx->ctx_lo + n_nodes > kAttLongContext ? 8 : 4;
  while (splits < cap && ctx->cfg.n_heads * ctx->batch * ntile * splits * 2 <= 296) splits *= 2;
  return splits;
}

// Batches whose (head, sequence) items alone fill the device go through the persistent page-stream kernel.
bool attention_streams(const vadusa_ctx* ctx, int n_nodes) {
  const vadusa_config& c = ctx->cfg;
  return ctx->att_stream && c.dtype == 1 && c.d_model / c.n_heads == 64 && n_nodes <= 64 && ctx->batch <= kAsMaxBatch &&
         attention_splits(ctx, n_nodes) == 1 && (long long)c.max_blocks_per_seq * kKvBlock < (1ll << 24);
}

template <typename T>
vadusa_status attention(vadusa_ctx* ctx, const T* q, const T* pool, const TreeView& tv, T* out) {
  const vadusa_config& c = ctx->cfg;
  const int dh = c.d_model / c.n_heads;
  const KvGeom g = geom_of(ctx);
  const float scale = (float)(1.0 / sqrt((double)dh));
  const int ntile = (tv.n_nodes + 63) / 64;
  dim3 grid(c.n_heads, ctx->batch * ntile);
  const size_t smem = (size_t)(64 * dh * 3 + 64 + 64 * 64) * sizeof(float);   // = attention_smem(dh)
  auto go = [&](auto kern) -> vadusa_status {
    PROF(ctx, K_ATTENTION);
    kern<<<grid, 256, smem, ctx->stream>>>(q, pool, ctx->block_table, wsptr<int32_t>(ctx, ctx->ws.ctx_len),
                                           wsptr<int32_t>(ctx, ctx->ws.nvalid), tv, g, c.d_model, scale, out,
                                           err_word(ctx));
    LAUNCH_CHECK();
    return VADUSA_OK;
  };
  if constexpr (std::is_same<T, bf16>::value) {
    if (dh == 64) {
      if (ctx->pf_tiles > 0 && tv.n_nodes == 64) {
        // prefill pass: two consecutive chunks of a sequence per CTA (128 query rows per K/V page fetched)
        const CUtensorMap *mq, *mkv;
        const int M = ctx->batch * tv.n_nodes;
        if (vadusa_status s = tensor_map(ctx, q, M, c.d_model, 64, 1, 0, &mq)) return s;
        const long long rows = (long long)c.kv_num_blocks * 2 * c.n_heads * kKvBlock;
        if (rows > 0x7fffffffLL) return fail(ctx, VADUSA_EINVAL, "KV pool too large for one tensor map");
        if (vadusa_status s = tensor_map(ctx, c.kv_pool, (int)rows, 64, 64, c.n_layers, g.layer_stride, &mkv)) return s;
        const int layer = (int)((reinterpret_cast<const char*>(pool) - reinterpret_cast<const char*>(c.kv_pool)) /
                                (g.layer_stride * (long long)sizeof(bf16)));
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(c.n_heads, ctx->pf_tiles, 1);
        lc.blockDim = dim3(kPfThreads);
        lc.dynamicSmemBytes = kAttSmemBytes;
        lc.stream = ctx->stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at; lc.numAttrs = 1;
        PROF(ctx, K_ATTENTION);
        CU(cudaLaunchKernelEx(&lc, prefill_attention_tc_kernel, *mq, *mkv, layer, ctx->block_table,
                              (const int32_t*)wsptr<int32_t>(ctx, ctx->ws.ctx_len),
                              (const int32_t*)wsptr<int32_t>(ctx, ctx->ws.nvalid),
                              (const int2*)wsptr<int2>(ctx, ctx->ws.pf_pairs), g, c.d_model,
                              scale * 1.4426950408889634f, reinterpret_cast<bf16*>(out), err_word(ctx)));
        LAUNCH_CHECK();
        return VADUSA_OK;
      }
      // tensor-core kernel; KV splits so that about two CTAs per SM exist even at batch 1
      const int splits = attention_splits(ctx, tv.n_nodes);
      const CUtensorMap *mq, *mkv;
      const int M = ctx->batch * tv.n_nodes;
      if (vadusa_status s = tensor_map(ctx, q, M, c.d_model, 64, 1, 0, &mq)) return s;
      const long long rows = (long long)c.kv_num_blocks * 2 * c.n_heads * kKvBlock;
      if (rows > 0x7fffffffLL) return fail(ctx, VADUSA_EINVAL, "KV pool too large for one tensor map");
      if (vadusa_status s = tensor_map(ctx, c.kv_pool, (int)rows, 64, 64, c.n_layers, g.layer_stride, &mkv)) return s;
      const int layer = (int)((reinterpret_cast<const char*>(pool) - reinterpret_cast<const char*>(c.kv_pool)) /
                              (g.layer_stride * (long long)sizeof(bf16)));
      if (attention_streams(ctx, tv.n_nodes)) {
        // batches: every CTA takes an equal share of the stream of K/V pages of all (sequence, head) items
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(kAsGrid);
        lc.blockDim = dim3(kAsThreads);
        lc.dynamicSmemBytes = kAsSmemBytes;
        lc.stream = ctx->stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at; lc.numAttrs = 1;
        PROF(ctx, K_ATTENTION);
        CU(cudaLaunchKernelEx(&lc, tree_attention_stream_kernel, *mq, *mkv, layer, ctx->block_table,
                              (const int32_t*)wsptr<int32_t>(ctx, ctx->ws.ctx_len),
                              (const int32_t*)wsptr<int32_t>(ctx, ctx->ws.nvalid), tv, g, ctx->batch, c.d_model,
                              scale * 1.4426950408889634f, reinterpret_cast<bf16*>(out),
                              wsptr<float>(ctx, ctx->ws.att_xch), wsptr<uint32_t>(ctx, ctx->ws.att_cnt), err_word(ctx)));
        LAUNCH_CHECK();
        return VADUSA_OK;
      }
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3(c.n_heads, ctx->batch * ntile, splits);
      lc.blockDim = dim3(kAttThreads);
      lc.dynamicSmemBytes = kAttSmemBytes;
      lc.stream = ctx->stream;
      cudaLaunchAttribute at[2];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = splits;
      at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[1].val.programmaticStreamSerializationAllowed = 1;
      lc.attrs = at; lc.numAttrs = 2;
      PROF(ctx, K_ATTENTION);
      CU(cudaLaunchKernelEx(&lc, tree_attention_tc_kernel, *mq, *mkv, layer, ctx->block_table,
                            (const int32_t*)wsptr<int32_t>(ctx, ctx->ws.ctx_len),
                            (const int32_t*)wsptr<int32_t>(ctx, ctx->ws.nvalid),
                            (const int32_t*)(ctx->batch > 1 ? wsptr<int32_t>(ctx, ctx->ws.seq_order) : nullptr), tv, g, c.d_model,
                            scale * 1.4426950408889634f, splits, reinterpret_cast<bf16*>(out),
                            wsptr<float>(ctx, ctx->ws.att_xch), err_word(ctx)));
      LAUNCH_CHECK();
      return VADUSA_OK;
    }
  }
  if (dh == 64) return go(tree_attention_simt_kernel<T, 64>);
  return go(tree_attention_simt_kernel<T, 32>);
}

template <typename T>
vadusa_status layernorm(vadusa_ctx* ctx, const float* x, const float* g, const float* b, T* y, int rows) {
  const int d = ctx->cfg.d_model;
  const bool by_warp = rows >= 64 && d % 128 == 0 && d <= 2048;   // many rows: one warp per row
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(by_warp ? (rows + 7) / 8 : rows);
  lc.blockDim = dim3(256);
  lc.stream = ctx->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;       // the kernel calls griddepcontrol.wait
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = 1;
  PROF(ctx, K_LAYERNORM);
  if (by_warp) CU(cudaLaunchKernelEx(&lc, layernorm_rows_kernel<T>, x, g, b, y, rows, d, ctx->cfg.ln_eps));
  else CU(cudaLaunchKernelEx(&lc, layernorm_kernel<T>, x, g, b, y, rows, d, ctx->cfg.ln_eps));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// Can this pass run as the single persistent kernel?  One sequence of at most 64 nodes, bf16, head_dim 64,
// 8 or 16 heads (one cluster per head), feed-forward width in whole 128-row blocks per cluster (at most two),
// and a device that holds all clusters at once (asked when the kernel is first wanted).
bool fused_shape_ok(const vadusa_ctx* ctx, const TreeView& tv) {
  const vadusa_config& c = ctx->cfg;
  if (!ctx->fused_enabled || c.dtype != 1 || ctx->batch != 1 || tv.n_nodes > 64) return false;
  const int H = c.n_heads, d = c.d_model, F = c.d_ffn;
  if (d != 64 * H || (H != 8 && H != 16)) return false;
  if (F % (128 * H) || F / H > 256) return false;
  if ((ctx->ctx_bound + 64) / kKvBlock / 6 + 1 > kFfMaxPages) return false;
  if (c.n_layers > 1) {
    // the per-layer tensors must repeat at a constant stride (they do in the blob this library lays out)
    const long long st = find(ctx, "l1.wqkv")->offset - find(ctx, "l0.wqkv")->offset;
    if (st % 16) return false;
  }
  return true;
}

template <int CS>
vadusa_status fused_launch(vadusa_ctx* ctx, bool query_only, int* clusters, const CUtensorMap* const* maps, const FusedArgs* a) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(CS * ctx->cfg.n_heads);
  lc.blockDim = dim3(kFfThreads);
  lc.dynamicSmemBytes = FfCfg<CS>::kSmemBytes;
  lc.stream = ctx->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  if (query_only) {
    lc.numAttrs = 1;
    CU(cudaFuncSetAttribute(fused_forward_kernel<CS>, cudaFuncAttributeMaxDynamicSharedMemorySize, FfCfg<CS>::kSmemBytes));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, fused_forward_kernel<CS>, &lc) != cudaSuccess) { cudaGetLastError(); n = 0; }
    *clusters = n;
    return VADUSA_OK;
  }
  lc.numAttrs = 2;
  PROF(ctx, K_FUSED);
  CU(cudaLaunchKernelEx(&lc, fused_forward_kernel<CS>, *maps[0], *maps[1], *maps[2], *maps[3], *maps[4], *maps[5], *maps[6], *maps[7], *a));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

vadusa_status fused_forward(vadusa_ctx* ctx, const TreeView& tv, const int32_t* override_tokens, bf16* attn_tap, bool* launched) {
  *launched = false;
  const vadusa_config& c = ctx->cfg;
  const int H = c.n_heads, d = c.d_model, F = c.d_ffn, L = c.n_layers, M = tv.n_nodes, vp = vpad(&c);
  if (ctx->fused_cs < 0) {
    // clusters of 8 where the device holds one per head at once, else clusters of 6
    int n8 = 0, n6 = 0;
    if (vadusa_status s = fused_launch<8>(ctx, true, &n8, nullptr, nullptr)) return s;
    if (vadusa_status s = fused_launch<6>(ctx, true, &n6, nullptr, nullptr)) return s;
    ctx->fused_cs = n8 >= H ? 8 : n6 >= H ? 6 : 0;
    ctx->fused_clusters = ctx->fused_cs == 8 ? n8 : n6;
    ctx->fused_n8 = n8; ctx->fused_n6 = n6;
  }
  int cs = ctx->fused_cs;
  if (ctx->fused_enabled == 8 && ctx->fused_n8 >= H) cs = 8;
  if (ctx->fused_enabled == 6 && ctx->fused_n6 >= H) cs = 6;
  if (cs == 0) return VADUSA_OK;                            // not all clusters fit at once: the caller takes the other path
  const long long lstride = L > 1 ? find(ctx, "l1.wqkv")->offset - find(ctx, "l0.wqkv")->offset : 0;
  const LayerW& w0 = ctx->layers[0];
  const KvGeom g = geom_of(ctx);
  const CUtensorMap* maps[8];
  if (vadusa_status s = tensor_map(ctx, w0.wqkv, 3 * d, d, 64, L, lstride / 2, &maps[0])) return s;
  if (vadusa_status s = tensor_map(ctx, w0.wo, d, d, 64, L, lstride / 2, &maps[1])) return s;
  if (vadusa_status s = tensor_map(ctx, w0.w1, F, d, 128, L, lstride / 2, &maps[2])) return s;
  if (vadusa_status s = tensor_map(ctx, w0.w2, d, F, 64, L, lstride / 2, &maps[3])) return s;
  if (vadusa_status s = tensor_map(ctx, ctx->lm, vp, d, 128, 1, 0, &maps[4])) return s;
  if (vadusa_status s = tensor_map(ctx, ctx->wsp + ctx->ws.o, M, d, 64, 1, 0, &maps[5])) return s;
  if (vadusa_status s = tensor_map(ctx, ctx->wsp + ctx->ws.mid, M, F, 64, 1, 0, &maps[6])) return s;
  const long long rows = (long long)c.kv_num_blocks * 2 * c.n_heads * kKvBlock;
  if (rows > 0x7fffffffLL) return fail(ctx, VADUSA_EINVAL, "KV pool too large for one tensor map");
  if (vadusa_status s = tensor_map(ctx, c.kv_pool, (int)rows, 64, 64, c.n_layers, g.layer_stride, &maps[7])) return s;
  FusedArgs a;
  memset(&a, 0, sizeof(a));
  a.L = L; a.d = d; a.H = H; a.F = F; a.vocab = c.vocab; a.vpad = vp; a.n_phonemes = c.n_phonemes; a.max_pos = c.max_pos; a.M = M;
  a.eps = c.ln_eps;
  a.scale_log2e = (float)(1.0 / sqrt(64.0)) * 1.4426950408889634f;
  a.ln1_g = w0.ln1_g; a.ln1_b = w0.ln1_b; a.bqkv = w0.bqkv; a.bo = w0.bo; a.ln2_g = w0.ln2_g; a.ln2_b = w0.ln2_b;
  a.b1 = w0.b1; a.b2 = w0.b2;
  a.layer_stride = lstride;
  a.lnf_g = ctx->lnf_g; a.lnf_b = ctx->lnf_b;
  a.emb_audio = as<bf16>(ctx->emb_audio); a.emb_phon = as<bf16>(ctx->emb_phon); a.pos = as<bf16>(ctx->pos);
  a.xa = wsptr<float>(ctx, ctx->ws.x); a.xb = wsptr<float>(ctx, ctx->ws.f_xb);
  a.stats_a = wsptr<float2>(ctx, ctx->ws.f_stats_a); a.stats_b = wsptr<float2>(ctx, ctx->ws.f_stats_b);
  a.o = wsptr<bf16>(ctx, ctx->ws.o); a.mid = wsptr<bf16>(ctx, ctx->ws.mid); a.hfinal = wsptr<bf16>(ctx, ctx->ws.hfinal);
  a.logits = wsptr<float>(ctx, ctx->ws.logits);
  a.attn_tap = attn_tap;
  a.tokens = wsptr<int32_t>(ctx, ctx->ws.tokens);
  a.kv_row = wsptr<long long>(ctx, ctx->ws.kv_row);
  a.override_tokens = override_tokens;
  a.root = wsptr<int32_t>(ctx, ctx->ws.root); a.topk = wsptr<int32_t>(ctx, ctx->ws.topk);
  a.n_draft_heads = c.n_draft_heads; a.draft_topk = c.draft_topk;
  a.ctx_len = wsptr<int32_t>(ctx, ctx->ws.ctx_len); a.nvalid = wsptr<int32_t>(ctx, ctx->ws.nvalid);
  a.block_table = ctx->block_table;
  a.tree = tv; a.geom = g;
  a.kv_pool = reinterpret_cast<bf16*>(c.kv_pool);
  a.sync = wsptr<uint32_t>(ctx, ctx->ws.f_sync);
  a.err = err_word(ctx);
  vadusa_status s = cs == 8 ? fused_launch<8>(ctx, false, nullptr, maps, &a) : fused_launch<6>(ctx, false, nullptr, maps, &a);
  if (s) return s;
  *launched = true;
  return VADUSA_OK;
}

// One forward pass of the base model over batch * tv.n_nodes rows (verify step).
template <typename T>
vadusa_status forward(vadusa_ctx* ctx, const TreeView& tv, const int32_t* override_tokens, T* attn_tap) {
  const vadusa_config& c = ctx->cfg;
  const int B = ctx->batch, N = tv.n_nodes, M = B * N, d = c.d_model, f = c.d_ffn, vp = vpad(&c);
  const KvGeom g = geom_of(ctx);
  if constexpr (std::is_same<T, bf16>::value) {
    if (fused_shape_ok(ctx, tv)) {
      bool launched = false;
      if (vadusa_status s = fused_forward(ctx, tv, override_tokens, attn_tap, &launched)) return s;
      if (launched) return VADUSA_OK;
    }
  }
  float* x = wsptr<float>(ctx, ctx->ws.x);
  T* a = wsptr<T>(ctx, ctx->ws.a);
  T* q = wsptr<T>(ctx, ctx->ws.q);
  T* o = wsptr<T>(ctx, ctx->ws.o);
  T* mid = wsptr<T>(ctx, ctx->ws.mid);
  T* hfinal = wsptr<T>(ctx, ctx->ws.hfinal);
  float* logits = wsptr<float>(ctx, ctx->ws.logits);
  int32_t* ctx_len = wsptr<int32_t>(ctx, ctx->ws.ctx_len);
  int32_t* nvalid = wsptr<int32_t>(ctx, ctx->ws.nvalid);

  // LayerNorm statistics for the products that normalise their own operand (bf16 models, few tokens): left by
  // the embedding kernel and by the residual products
  const bool tc = std::is_same<T, bf16>::value;
  const bool embed_stats = tc && M <= 64 && d % 128 == 0 && d / 128 <= 8;
  const bool stats_out = tc && residual_leaves_stats(M, d, d), stats_ffn = tc && residual_leaves_stats(M, d, f);
  float2* stats = wsptr<float2>(ctx, ctx->ws.ln_stats);
  PROF(ctx, K_EMBED);
  tree_embed_kernel<T><<<M, 128, 0, ctx->stream>>>(
      tv, override_tokens, wsptr<int32_t>(ctx, ctx->ws.root), wsptr<int32_t>(ctx, ctx->ws.topk), c.n_draft_heads,
      c.draft_topk, ctx_len, nvalid, as<T>(ctx->emb_audio), as<T>(ctx->emb_phon), as<T>(ctx->pos),
      c.vocab, c.n_phonemes, c.max_pos, d, wsptr<int32_t>(ctx, ctx->ws.tokens), x, ctx->block_table, g,
      wsptr<long long>(ctx, ctx->ws.kv_row), embed_stats ? stats : nullptr, err_word(ctx));
  LAUNCH_CHECK();
  if (B > 1) {
    PROF(ctx, K_MISC);
    seq_order_kernel<<<1, 256, 0, ctx->stream>>>(ctx_len, nvalid, B, wsptr<int32_t>(ctx, ctx->ws.seq_order));
    LAUNCH_CHECK();
  }
  bool have_stats = embed_stats;
  for (int l = 0; l < c.n_layers; ++l) {
    const LayerW& w = ctx->layers[l];
    T* pool = reinterpret_cast<T*>(c.kv_pool) + (long long)l * g.layer_stride;
    vadusa_status s = VADUSA_OK;
    EpiQKV<T> eq{w.bqkv, q, pool, wsptr<long long>(ctx, ctx->ws.kv_row), (long long)c.n_heads * kKvBlock * g.head_dim,
                 kKvBlock * g.head_dim, g.head_dim, d};
    if (!(have_stats && ln_product<T>(ctx, K_GEMM_QKV, x, w.ln1_g, w.ln1_b, as<T>(w.wqkv), 3 * d, M, 3 * d, d, eq, &s))) {
      s = layernorm<T>(ctx, x, w.ln1_g, w.ln1_b, a, M);
      if (s) return s;
      s = product<T>(ctx, K_GEMM_QKV, a, as<T>(w.wqkv), 3 * d, M, 3 * d, d, 1, 0, 0, eq);
    }
    if (s) return s;
    s = attention<T>(ctx, q, pool, tv, o);
    if (s) return s;
    if (attn_tap)
      CU(cudaMemcpyAsync(attn_tap + (long long)l * M * d, o, (size_t)M * d * sizeof(T), cudaMemcpyDeviceToDevice, ctx->stream));
    if (stats_out) {
      EpiResidualStats eo{w.bo, x, d, stats};
      s = product<T>(ctx, K_GEMM_OUT, o, as<T>(w.wo), d, M, d, d, 1, 0, 0, eo);
      have_stats = true;
    } else {
      EpiResidual eo{w.bo, x, d};
      s = product<T>(ctx, K_GEMM_OUT, o, as<T>(w.wo), d, M, d, d, 1, 0, 0, eo);
    }
    if (s) return s;
    EpiRelu<T> e1{w.b1, mid, f};
    if (!(have_stats && ln_product<T>(ctx, K_GEMM_FFN1, x, w.ln2_g, w.ln2_b, as<T>(w.w1), f, M, f, d, e1, &s))) {
      s = layernorm<T>(ctx, x, w.ln2_g, w.ln2_b, a, M);
      if (s) return s;
      s = product<T>(ctx, K_GEMM_FFN1, a, as<T>(w.w1), f, M, f, d, 1, 0, 0, e1);
    }
    if (s) return s;
    if (stats_ffn) {
      EpiResidualStats e2{w.b2, x, d, stats};
      s = product<T>(ctx, K_GEMM_FFN2, mid, as<T>(w.w2), d, M, d, f, 1, 0, 0, e2);
    } else {
      EpiResidual e2{w.b2, x, d};
      s = product<T>(ctx, K_GEMM_FFN2, mid, as<T>(w.w2), d, M, d, f, 1, 0, 0, e2);
    }
    have_stats = stats_ffn;
    if (s) return s;
  }
  EpiLogits el{logits, vp, 0};
  vadusa_status s = VADUSA_OK;
  // the final LayerNorm folds into the vocabulary head, which also stores the normalised rows (the draft heads
  // and the carried state read them)
  if (have_stats && ln_product<T>(ctx, K_GEMM_LM, x, ctx->lnf_g, ctx->lnf_b, as<T>(ctx->lm), vp, M, vp, d, el, &s, hfinal))
    return s;
  if ((s = layernorm<T>(ctx, x, ctx->lnf_g, ctx->lnf_b, hfinal, M))) return s;
  return product<T>(ctx, K_GEMM_LM, hfinal, as<T>(ctx->lm), vp, M, vp, d, 1, 0, 0, el);
}

template <typename T>
vadusa_status draft(vadusa_ctx* ctx, const SamplingDev& sp) {
  const vadusa_config& c = ctx->cfg;
  const int B = ctx->batch, d = c.d_model, vp = vpad(&c), hd = c.n_draft_heads;
  const T* hstar = wsptr<T>(ctx, ctx->ws.hstar);
  T* z = wsptr<T>(ctx, ctx->ws.z);
  float* dl = wsptr<float>(ctx, ctx->ws.dlogits);
  const long long w_stride = ctx->dw_stride / (long long)sizeof(T), u_stride = ctx->du_stride / (long long)sizeof(T);
  if (hd > 1 && w_stride != (long long)d * d) return fail(ctx, VADUSA_EINVAL, "draft matrices are not contiguous");
  EpiDraftHiddenFlat<T> eh{ctx->db, hstar, z, d, B};
  vadusa_status s = product<T>(ctx, K_DRAFT_HIDDEN, hstar, as<T>(ctx->dw), hd * d, B, hd * d, d, 1, 0, 0, eh);
  if (s) return s;
  EpiLogits el{dl, vp, (long long)B * vp};
  s = product<T>(ctx, K_DRAFT_LOGITS, z, as<T>(ctx->du), vp, B, vp, d, hd, (long long)B * d, u_stride, el);
  if (s) return s;
  dim3 grid(hd + 1, B);
  PROF(ctx, K_DRAFT_SELECT);
  draft_select_kernel<<<grid, 256, 0, ctx->stream>>>(dl, wsptr<float>(ctx, ctx->ws.logits_star), vp, c.vocab, B, hd,
                                                     c.draft_topk, wsptr<int32_t>(ctx, ctx->ws.ctx_len),
                                                     wsptr<int32_t>(ctx, ctx->ws.nvalid), sp,
                                                     wsptr<int32_t>(ctx, ctx->ws.topk),
                                                     wsptr<int32_t>(ctx, ctx->ws.root));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// tokens = tree built from the draft (no model pass): used when the caller wants them.
template <typename T>
vadusa_status accept_commit(vadusa_ctx* ctx, const SamplingDev& sp, const int32_t* forced, const AcceptOut& out,
                            int32_t* out_tokens, int out_cap, int target) {
  const vadusa_config& c = ctx->cfg;
  const int B = ctx->batch, vp = vpad(&c);
  const KvGeom g = geom_of(ctx);
  const TreeView tv = tree_of(ctx, false);
  SeqState st = state_of(ctx, out_tokens, out_cap, target);
  PROF(ctx, K_ACCEPT);
  accept_kernel<<<B, 256, 2 * vp * sizeof(float), ctx->stream>>>(
      wsptr<float>(ctx, ctx->ws.logits), vp, c.vocab, wsptr<int32_t>(ctx, ctx->ws.tokens), tv, ctx->block_table, g,
      sp, forced, st, out, err_word(ctx));
  LAUNCH_CHECK();
  dim3 grid(c.n_layers + 1, B);
  PROF(ctx, K_COMMIT);
  commit_kernel<T><<<grid, 256, 0, ctx->stream>>>(
      reinterpret_cast<T*>(c.kv_pool), g, ctx->block_table, st, c.n_layers, tv.n_nodes,
      wsptr<T>(ctx, ctx->ws.hfinal), c.d_model, wsptr<float>(ctx, ctx->ws.logits), vp, wsptr<T>(ctx, ctx->ws.hstar),
      wsptr<float>(ctx, ctx->ws.logits_star), err_word(ctx));
  LAUNCH_CHECK();
  return VADUSA_OK;
}

// While alive, the model's passes see `rows` rows described by the given arrays instead of the batch.
struct RowsView {
  vadusa_ctx* c;
  int batch; const int32_t* table; int64_t ctx_len, nvalid;
  RowsView(vadusa_ctx* ctx, int rows, const int32_t* block_table, int64_t ctx_len_off, int64_t nvalid_off)
      : c(ctx), batch(ctx->batch), table(ctx->block_table), ctx_len(ctx->ws.ctx_len), nvalid(ctx->ws.nvalid) {
    ctx->batch = rows; ctx->block_table = block_table; ctx->ws.ctx_len = ctx_len_off; ctx->ws.nvalid = nvalid_off;
  }
  ~RowsView() { c->batch = batch; c->block_table = table; c->ws.ctx_len = ctx_len; c->ws.nvalid = nvalid; }
};

template <typename T>
vadusa_status prefill(vadusa_ctx* ctx, const int32_t* h_tokens, const int32_t* h_len, int stride) {
  const vadusa_config& c = ctx->cfg;
  const int B = ctx->batch, N = c.max_tree_nodes, vp = vpad(&c), R = pass_rows(&c);
  int longest = 0;
  for (int b = 0; b < B; ++b) {
    if (h_len[b] < 1 || h_len[b] > stride) return fail(ctx, VADUSA_EINVAL, "prefix length of sequence %d out of range", b);
    longest = h_len[b] > longest ? h_len[b] : longest;
  }
  // what the cache holds already
  std::vector<int32_t> base(B);
  CU(cudaMemcpyAsync(base.data(), ctx->wsp + ctx->ws.ctx_len, B * sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  // chunks in sequence order, so that a chunk never precedes an earlier chunk of its sequence
  struct Chunk { int b, s0, n, last; };
  std::vector<Chunk> chunks;
  for (int b = 0; b < B; ++b)
    for (int s0 = 0; s0 < h_len[b]; s0 += N) {
      const int n = h_len[b] - s0 < N ? h_len[b] - s0 : N;
      chunks.push_back({b, s0, n, s0 + n == h_len[b] ? b : -1});
    }
  int32_t* d_stage = wsptr<int32_t>(ctx, ctx->ws.stage_tokens);
  int32_t* d_ctx = wsptr<int32_t>(ctx, ctx->ws.pf_ctx_len);
  int32_t* d_nv = wsptr<int32_t>(ctx, ctx->ws.pf_nvalid);
  int32_t* d_seq = wsptr<int32_t>(ctx, ctx->ws.pf_seq);
  int32_t* d_last = wsptr<int32_t>(ctx, ctx->ws.pf_last);
  int32_t* d_table = wsptr<int32_t>(ctx, ctx->ws.pf_block_table);
  int32_t* real_ctx_len = wsptr<int32_t>(ctx, ctx->ws.ctx_len);
  const int32_t* real_table = ctx->block_table;
  std::vector<int32_t> stage((size_t)R * N), v_ctx(R), v_nv(R), v_seq(R), v_last(R), v_pairs(2 * (size_t)R);
  const TreeView tv = tree_of(ctx, true);
  for (size_t c0 = 0; c0 < chunks.size(); c0 += R) {
    const int rows = (int)(chunks.size() - c0 < (size_t)R ? chunks.size() - c0 : R);
    for (int r = 0; r < rows; ++r) {
      const Chunk& ch = chunks[c0 + r];
      v_ctx[r] = base[ch.b] + ch.s0; v_nv[r] = ch.n; v_seq[r] = ch.b; v_last[r] = ch.last;
      for (int i = 0; i < N; ++i) stage[(size_t)r * N + i] = i < ch.n ? h_tokens[(size_t)ch.b * stride + ch.s0 + i] : 0;
    }
    CU(cudaMemcpyAsync(d_ctx, v_ctx.data(), rows * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(d_nv, v_nv.data(), rows * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(d_seq, v_seq.data(), rows * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(d_last, v_last.data(), rows * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(d_stage, stage.data(), (size_t)rows * N * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
    // attention tiles of the pass: a full chunk and the chunk behind it in the same sequence share a CTA
    int tiles = 0;
    for (int r = 0; r < rows;) {
      const Chunk& ch = chunks[c0 + r];
      const bool pair = r + 1 < rows && chunks[c0 + r + 1].b == ch.b && ch.n == N;
      v_pairs[2 * tiles] = r; v_pairs[2 * tiles + 1] = pair ? r + 1 : -1;
      ++tiles;
      r += pair ? 2 : 1;
    }
    CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.pf_pairs, v_pairs.data(), (size_t)tiles * 8, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));   // the staging vectors are reused by the next pass
    prefill_gather_kernel<<<rows, 128, 0, ctx->stream>>>(real_table, d_seq, c.max_blocks_per_seq, d_table);
    LAUNCH_CHECK();
    {
      RowsView view(ctx, rows, d_table, ctx->ws.pf_ctx_len, ctx->ws.pf_nvalid);
      ctx->pf_tiles = tiles;
      const vadusa_status s = forward<T>(ctx, tv, d_stage, nullptr);
      ctx->pf_tiles = 0;
      if (s) return s;
    }
    prefill_finish_kernel<T><<<rows, 256, 0, ctx->stream>>>(d_ctx, d_nv, d_last, N, wsptr<T>(ctx, ctx->ws.hfinal), c.d_model,
                                                            wsptr<float>(ctx, ctx->ws.logits), vp,
                                                            wsptr<T>(ctx, ctx->ws.hstar),
                                                            wsptr<float>(ctx, ctx->ws.logits_star), real_ctx_len);
    LAUNCH_CHECK();
    if (ctx->pf_tap)
      for (int r = 0; r < rows; ++r) {
        const Chunk& ch = chunks[c0 + r];
        if (ch.s0 + ch.n > ctx->pf_tap_stride) return fail(ctx, VADUSA_EINVAL, "prefill tap: row stride shorter than the prefix");
        CU(cudaMemcpyAsync(reinterpret_cast<T*>(ctx->pf_tap) + ((long long)ch.b * ctx->pf_tap_stride + ch.s0) * c.d_model,
                           wsptr<T>(ctx, ctx->ws.hfinal) + (long long)r * N * c.d_model, (size_t)ch.n * c.d_model * sizeof(T),
                           cudaMemcpyDeviceToDevice, ctx->stream));
      }
  }
  ctx->ctx_bound += longest;
  ctx->ctx_lo += longest;
  CU(cudaStreamSynchronize(ctx->stream));
  return VADUSA_OK;
}

// ---- draft-head fitting -------------------------------------------------------------------
struct FitLayout {
  int64_t W, b, U, n_params;               // fp32 masters, contiguous: [heads][d][d], [heads][d], [heads][vpad][d]
  int64_t m, v, g;                         // Adam moments and gradients, same shape as the masters
  int64_t hf, pre, z, dz, logits, ce, count, total;
};
FitLayout fit_layout(const vadusa_config* c, int max_tokens) {
  FitLayout f;
  const int64_t hd = c->n_draft_heads, d = c->d_model, vp = vpad(c), T = max_tokens;
  int64_t off = 0;
  auto take = [&](int64_t bytes) { int64_t o = off; off = align_up(off + bytes, 256); return o; };
  f.n_params = hd * (d * d + d + vp * d);
  f.W = take(f.n_params * 4); f.b = f.W + hd * d * d * 4; f.U = f.b + hd * d * 4;
  f.m = take(f.n_params * 4); f.v = take(f.n_params * 4); f.g = take(f.n_params * 4);
  f.hf = take(T * d * 4); f.pre = take(hd * T * d * 4); f.z = take(hd * T * d * 4); f.dz = take(hd * T * d * 4);
  f.logits = take(hd * T * vp * 4); f.ce = take(hd * T * 4); f.count = take(hd * 4);
  f.total = off;
  return f;
}

template <typename T>
vadusa_status fit_begin(vadusa_ctx* ctx, const FitLayout& f) {
  const vadusa_config& c = ctx->cfg;
  const long long hd = c.n_draft_heads, d = c.d_model, vp = vpad(&c);
  auto up = [&](const T* src, int64_t off, long long n) -> vadusa_status {
    fit_to_f32_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, ctx->stream>>>(src, reinterpret_cast<float*>(ctx->fit + off), n);
    LAUNCH_CHECK();
    return VADUSA_OK;
  };
  if (vadusa_status s = up(as<T>(ctx->dw), f.W, hd * d * d)) return s;
  if (vadusa_status s = up(as<T>(ctx->du), f.U, hd * vp * d)) return s;
  CU(cudaMemcpyAsync(ctx->fit + f.b, ctx->db, (size_t)(hd * d * 4), cudaMemcpyDeviceToDevice, ctx->stream));
  CU(cudaMemsetAsync(ctx->fit + f.m, 0, (size_t)(f.n_params * 4), ctx->stream));
  CU(cudaMemsetAsync(ctx->fit + f.v, 0, (size_t)(f.n_params * 4), ctx->stream));
  return VADUSA_OK;
}

template <typename T>
vadusa_status fit_step(vadusa_ctx* ctx, const FitLayout& f, const T* hidden, const int32_t* targets, int Tn, float* loss_out) {
  const vadusa_config& c = ctx->cfg;
  const int hd = c.n_draft_heads, d = c.d_model, vp = vpad(&c), V = c.vocab;
  auto P = [&](int64_t off) { return reinterpret_cast<float*>(ctx->fit + off); };
  float *W = P(f.W), *b = P(f.b), *U = P(f.U), *gW = P(f.g), *gb = gW + (long long)hd * d * d, *gU = gb + (long long)hd * d;
  float *hf = P(f.hf), *pre = P(f.pre), *z = P(f.z), *dz = P(f.dz), *lg = P(f.logits), *ce = P(f.ce);
  int32_t* count = reinterpret_cast<int32_t*>(ctx->fit + f.count);
  const long long hs = (long long)Tn * d, ls = (long long)Tn * vp;
  cudaStream_t st = ctx->stream;
  auto gemm = [&](const float* A, const float* B, float* C, int M, int N, int K, long long sam, long long sak, long long sbn,
                  long long sbk, long long ldc, long long az, long long bz, long long cz) -> vadusa_status {
    dim3 grid((N + 63) / 64, (M + 63) / 64, hd);
    fit_gemm_kernel<<<grid, 256, 0, st>>>(A, B, C, M, N, K, sam, sak, sbn, sbk, ldc, az, bz, cz);
    LAUNCH_CHECK();
    return VADUSA_OK;
  };
  const unsigned eb = (unsigned)((hs + 255) / 256);
  fit_to_f32_kernel<T><<<eb, 256, 0, st>>>(hidden, hf, hs);
  LAUNCH_CHECK();
  fit_count_kernel<<<1, 256, 0, st>>>(targets, Tn, hd, count);
  LAUNCH_CHECK();
  // forward: pre = h W^T (+ b), z = h + SiLU(pre), logits = z U^T
  if (vadusa_status s = gemm(hf, W, pre, Tn, d, d, d, 1, d, 1, d, 0, (long long)d * d, hs)) return s;
  fit_hidden_kernel<<<dim3(eb, hd), 256, 0, st>>>(pre, b, hf, z, Tn, d, hs);
  LAUNCH_CHECK();
  if (vadusa_status s = gemm(z, U, lg, Tn, vp, d, d, 1, d, 1, vp, hs, (long long)vp * d, ls)) return s;
  // loss and d loss / d logits (over the logits)
  fit_softmax_ce_kernel<<<dim3(Tn, hd), 256, 0, st>>>(lg, targets, count, Tn, hd, V, vp, ctx->fit_lambda, ce);
  LAUNCH_CHECK();
  fit_loss_kernel<<<1, 256, 0, st>>>(ce, count, Tn, hd, ctx->fit_lambda, loss_out);
  LAUNCH_CHECK();
  // backward: dU = dl^T z, dz = dl U, dpre = dz SiLU'(pre), dW = dpre^T h, db = column sums of dpre
  if (vadusa_status s = gemm(lg, z, gU, vp, d, Tn, 1, vp, 1, d, d, ls, hs, (long long)vp * d)) return s;
  if (vadusa_status s = gemm(lg, U, dz, Tn, d, vp, vp, 1, 1, d, d, ls, (long long)vp * d, hs)) return s;
  fit_dpre_kernel<<<dim3(eb, hd), 256, 0, st>>>(dz, pre, hs, hs);
  LAUNCH_CHECK();
  if (vadusa_status s = gemm(dz, hf, gW, d, d, Tn, 1, d, 1, d, d, hs, 0, (long long)d * d)) return s;
  fit_colsum_kernel<<<dim3((d + 255) / 256, hd), 256, 0, st>>>(dz, gb, Tn, d, hs);
  LAUNCH_CHECK();
  // update (Adam, linear warm-up), masters and the heads in the weight blob
  ctx->fit_step++;
  const float lr = ctx->fit_lr * fminf(1.0f, (float)ctx->fit_step / (float)(ctx->fit_warmup > 0 ? ctx->fit_warmup : 1));
  const float c1 = (float)(1.0 - pow(0.9, (double)ctx->fit_step)), c2 = (float)(1.0 - pow(0.999, (double)ctx->fit_step));
  float *mW = P(f.m), *vW = P(f.v);
  const long long nW = (long long)hd * d * d, nb = (long long)hd * d, nU = (long long)hd * vp * d;
  fit_adam_kernel<T><<<(unsigned)((nW + 255) / 256), 256, 0, st>>>(W, gW, mW, vW, const_cast<T*>(as<T>(ctx->dw)), nW, lr, c1, c2);
  LAUNCH_CHECK();
  fit_adam_kernel<float><<<(unsigned)((nb + 255) / 256), 256, 0, st>>>(b, gb, mW + nW, vW + nW, const_cast<float*>(ctx->db), nb, lr, c1, c2);
  LAUNCH_CHECK();
  fit_adam_kernel<T><<<(unsigned)((nU + 255) / 256), 256, 0, st>>>(U, gU, mW + nW + nb, vW + nW + nb, const_cast<T*>(as<T>(ctx->du)), nU, lr, c1, c2);
  LAUNCH_CHECK();
  return VADUSA_OK;
}

size_t attention_smem(int dh) { return (size_t)(64 * dh * 3 + 64 + 64 * 64) * sizeof(float); }

vadusa_status set_kernel_attributes(vadusa_ctx* ctx) {
  CU(cudaFuncSetAttribute(tree_attention_simt_kernel<float, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_smem(64)));
  CU(cudaFuncSetAttribute(tree_attention_simt_kernel<float, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_smem(32)));
  CU(cudaFuncSetAttribute(tree_attention_simt_kernel<bf16, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_smem(64)));
  CU(cudaFuncSetAttribute(tree_attention_simt_kernel<bf16, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_smem(32)));
  CU(cudaFuncSetAttribute(tree_attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmemBytes));
  CU(cudaFuncSetAttribute(prefill_attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmemBytes));
  CU(cudaFuncSetAttribute(tree_attention_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAsSmemBytes));
  CU(cudaFuncSetAttribute(prefill_attention_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
  // the accept kernel keeps one row of keys and one of probabilities in shared memory.  The limit is an attribute of
  // the function on this device, shared by every context: always the library's largest vocabulary
  CU(cudaFuncSetAttribute(accept_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 24576 * (int)sizeof(float)));
  // ask for the largest shared-memory carve-out so that several CTAs fit on an SM
  CU(cudaFuncSetAttribute(tree_attention_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
  CU(cudaFuncSetAttribute(tree_attention_stream_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
  return VADUSA_OK;
}

__global__ void fill_i32_kernel(int32_t* p, int n, int32_t v) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

vadusa_status set_active(vadusa_ctx* ctx, int value) {
  fill_i32_kernel<<<(ctx->batch + 255) / 256, 256, 0, ctx->stream>>>(wsptr<int32_t>(ctx, ctx->ws.nvalid), ctx->batch,
                                                                     value);
  LAUNCH_CHECK();
  return VADUSA_OK;
}

vadusa_status device_errors(vadusa_ctx* ctx) {
  uint32_t e = 0;
  CU(cudaMemcpyAsync(&e, err_word(ctx), sizeof(e), cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  if (e & kErrTimeout) return fail(ctx, VADUSA_ETIMEOUT, "a bounded device-side wait expired (error word 0x%x)", e);
  if (e & kErrCapacity)
    return fail(ctx, VADUSA_ECAPACITY, "a sequence ran past its KV blocks, the position table or the token range (error word 0x%x)", e);
  return VADUSA_OK;
}

// Key of a launch sequence: a tag plus the raw bytes of everything baked into its kernels' arguments.
struct KeyBuilder {
  std::string k;
  explicit KeyBuilder(const char* tag) : k(tag) {}
  template <typename V> KeyBuilder& add(const V& v) { k.append(reinterpret_cast<const char*>(&v), sizeof(V)); return *this; }
};

// Runs `body` (which only enqueues work on ctx->stream) eagerly the first time a key is seen,
// captures it into a CUDA graph the second time, and replays the graph afterwards.  The legacy
// default stream cannot be captured, and profiling wants separate launches: both run eagerly.
template <typename F>
vadusa_status run_graphed(vadusa_ctx* ctx, const std::string& key, F&& body) {
  if (ctx->stream == nullptr || ctx->prof_on) return body();
  if (ctx->graphs.size() > 64) {
    for (auto& kv : ctx->graphs) if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    ctx->graphs.clear();
  }
  vadusa_ctx::GraphRec& r = ctx->graphs[key];
  if (r.exec) {
    CU(cudaGraphLaunch(r.exec, ctx->stream));
    ctx->launches += r.launches;
    return VADUSA_OK;
  }
  if (r.seen++ == 0) return body();
  const int64_t l0 = ctx->launches;
  CU(cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
  vadusa_status s = body();
  cudaGraph_t graph = nullptr;
  cudaError_t ce = cudaStreamEndCapture(ctx->stream, &graph);
  if (s != VADUSA_OK || ce != cudaSuccess || !graph) {
    if (graph) cudaGraphDestroy(graph);
    cudaGetLastError();
    if (s != VADUSA_OK) return s;
    return fail(ctx, VADUSA_ECUDA, "stream capture failed: %s", cudaGetErrorString(ce));
  }
  ce = cudaGraphInstantiate(&r.exec, graph, 0);
  cudaGraphDestroy(graph);
  if (ce != cudaSuccess) { r.exec = nullptr; return fail(ctx, VADUSA_ECUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(ce)); }
  r.launches = ctx->launches - l0;
  ctx->launches = l0;
  CU(cudaGraphLaunch(r.exec, ctx->stream));
  ctx->launches += r.launches;
  return VADUSA_OK;
}

#define DISPATCH(expr_f32, expr_bf16) (ctx->cfg.dtype == 1 ? (expr_bf16) : (expr_f32))

vadusa_status need_batch(vadusa_ctx* ctx) {
  if (!ctx) return VADUSA_EINVAL;
  if (ctx->batch == 0) return fail(ctx, VADUSA_ESTATE, "vadusa_begin has not been called");
  return VADUSA_OK;
}

}  // namespace

// ---- C ABI -------------------------------------------------------------------------

extern "C" {

int64_t vadusa_workspace_bytes(const vadusa_config* cfg) {
  if (check_config(cfg)) return -1;
  return workspace_layout(cfg).total;
}

int64_t vadusa_weights_bytes(const vadusa_config* cfg) {
  if (check_config(cfg)) return -1;
  int64_t total = 0;
  weight_layout(cfg, &total);
  return total;
}

int64_t vadusa_kv_pool_bytes(const vadusa_config* cfg) {
  if (check_config(cfg)) return -1;
  return kv_pool_bytes(cfg);
}

int32_t vadusa_weight_count(const vadusa_config* cfg) {
  if (check_config(cfg)) return -1;
  return (int32_t)weight_layout(cfg, nullptr).size();
}

vadusa_status vadusa_weight_info(const vadusa_config* cfg, int32_t index, vadusa_tensor_info* h_out) {
  if (check_config(cfg) || !h_out) return VADUSA_EINVAL;
  auto v = weight_layout(cfg, nullptr);
  if (index < 0 || index >= (int32_t)v.size()) return VADUSA_EINVAL;
  const TensorDesc& t = v[index];
  memset(h_out, 0, sizeof(*h_out));
  snprintf(h_out->name, sizeof(h_out->name), "%s", t.name.c_str());
  h_out->offset = t.offset; h_out->nbytes = t.nbytes;
  h_out->rows = t.rows; h_out->cols = t.cols; h_out->rows_padded = t.rows_padded; h_out->is_matrix = t.is_matrix;
  return VADUSA_OK;
}

vadusa_status vadusa_init(const vadusa_weights* weights, const vadusa_config* cfg, vadusa_ctx** h_out) {
  if (!h_out) return VADUSA_EINVAL;
  *h_out = nullptr;
  vadusa_ctx* ctx = new (std::nothrow) vadusa_ctx();
  if (!ctx) return VADUSA_ENOMEM;
  *h_out = ctx;     // returned even on failure so that vadusa_last_error can be read; destroy it either way
  if (const char* why = check_config(cfg)) return fail(ctx, VADUSA_EINVAL, "%s", why);
  ctx->cfg = *cfg;
  if (!weights || !weights->blob) return fail(ctx, VADUSA_EINVAL, "weights are NULL");
  int64_t wbytes = 0;
  ctx->wl = weight_layout(cfg, &wbytes);
  if (weights->nbytes < wbytes) return fail(ctx, VADUSA_ENOMEM, "weight blob has %lld bytes, %lld needed", (long long)weights->nbytes, (long long)wbytes);
  ctx->ws = workspace_layout(cfg);
  if (!cfg->workspace || cfg->workspace_bytes < ctx->ws.total)
    return fail(ctx, VADUSA_ENOMEM, "workspace has %lld bytes, %lld needed", (long long)cfg->workspace_bytes, (long long)ctx->ws.total);
  if (((uintptr_t)cfg->workspace & 255) || ((uintptr_t)weights->blob & 255) || ((uintptr_t)cfg->kv_pool & 255))
    return fail(ctx, VADUSA_EINVAL, "workspace, weight blob and KV pool must be 256-byte aligned");
  if (!cfg->kv_pool || cfg->kv_pool_bytes < kv_pool_bytes(cfg))
    return fail(ctx, VADUSA_ENOMEM, "KV pool has %lld bytes, %lld needed", (long long)cfg->kv_pool_bytes, (long long)kv_pool_bytes(cfg));
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    return fail(ctx, VADUSA_ECUDA, "no CUDA device: this library has no CPU path");
  }
  if (cfg->device < 0 || cfg->device >= ndev) return fail(ctx, VADUSA_EINVAL, "device ordinal out of range");
  CU(cudaSetDevice(cfg->device));
  cudaDeviceProp prop;
  CU(cudaGetDeviceProperties(&prop, cfg->device));
  if (prop.major != 10) return fail(ctx, VADUSA_ECUDA, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
  ctx->blob = reinterpret_cast<const char*>(weights->blob);
  ctx->wsp = reinterpret_cast<char*>(cfg->workspace);
  ctx->stream = reinterpret_cast<cudaStream_t>(cfg->stream);
  resolve_weights(ctx);
  {
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      ctx->encode_fn = fn;
    else
      cudaGetLastError();
  }
  if (vadusa_status s = set_kernel_attributes(ctx)) return s;
  CU(cudaEventCreate(&ctx->ev0));
  CU(cudaEventCreate(&ctx->ev1));
  CU(cudaEventCreateWithFlags(&ctx->ev_poll, cudaEventDisableTiming));
  CU(cudaMallocHost(&ctx->h_pinned, 4 * sizeof(int32_t)));
  CU(cudaMemsetAsync(ctx->wsp, 0, ctx->ws.tokens, ctx->stream));     // scalars, per-sequence state, trees
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.acc_stats, 0, 2ull * kStatDepth * kStatTopk * 8, ctx->stream));
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.f_sync, 0, 256, ctx->stream));
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.att_cnt, 0, 2 * kAsGrid * 4, ctx->stream));
  // chain-shaped tree used by prefill: node i is the child of node i-1
  constexpr int T = VADUSA_MAX_TREE_NODES;
  static_assert(T == kMaxNodes, "node limit of the kernels");
  int32_t par[T], dep[T], rnk[T];
  unsigned long long anc[2 * T];
  auto low_bits = [](int n) { return n <= 0 ? 0ull : n >= 64 ? ~0ull : ((1ull << n) - 1); };   // n lowest bits set
  for (int i = 0; i < T; ++i) { par[i] = i - 1; dep[i] = i; rnk[i] = 0; anc[2 * i] = low_bits(i + 1); anc[2 * i + 1] = low_bits(i + 1 - 64); }
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.chain_parent, par, sizeof(par), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.chain_depth, dep, sizeof(dep), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.chain_rank, rnk, sizeof(rnk), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.chain_anc, anc, sizeof(anc), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return VADUSA_OK;
}

vadusa_status vadusa_destroy(vadusa_ctx* ctx) {
  if (!ctx) return VADUSA_EINVAL;
  if (ctx->ev0) cudaEventDestroy(ctx->ev0);
  if (ctx->ev1) cudaEventDestroy(ctx->ev1);
  if (ctx->ev_poll) cudaEventDestroy(ctx->ev_poll);
  if (ctx->h_pinned) cudaFreeHost(ctx->h_pinned);
  for (auto& r : ctx->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  for (auto& kv : ctx->graphs) if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
  delete ctx;
  return VADUSA_OK;
}

const char* vadusa_last_error(const vadusa_ctx* ctx) { return ctx ? ctx->err : "context is NULL"; }

vadusa_status vadusa_set_tree(vadusa_ctx* ctx, int32_t n_nodes, const int32_t* h_parent, const int32_t* h_rank,
                              int32_t per_sequence) {
  if (!ctx) return VADUSA_EINVAL;
  if (!ctx->wsp) return fail(ctx, VADUSA_ESTATE, "context is not initialised");
  if (!h_parent || !h_rank) return fail(ctx, VADUSA_EINVAL, "tree arrays are NULL");
  if (n_nodes < 1 || n_nodes > ctx->cfg.max_tree_nodes) return fail(ctx, VADUSA_EINVAL, "n_nodes must be in 1..max_tree_nodes");
  int copies = 1;
  if (per_sequence) {
    if (ctx->batch == 0) return fail(ctx, VADUSA_ESTATE, "per-sequence trees need vadusa_begin first");
    copies = ctx->batch;
  }
  std::vector<int32_t> depth((size_t)copies * n_nodes);
  std::vector<unsigned long long> anc((size_t)copies * n_nodes * 2);
  int max_rank = 0, max_depth = 0;
  for (int s = 0; s < copies; ++s) {
    const int32_t* par = h_parent + (size_t)s * n_nodes;
    const int32_t* rnk = h_rank + (size_t)s * n_nodes;
    int32_t* dep = depth.data() + (size_t)s * n_nodes;
    unsigned long long* an = anc.data() + (size_t)s * n_nodes * 2;       // two words per node
    if (par[0] != -1) return fail(ctx, VADUSA_EINVAL, "node 0 must be the root (parent -1)");
    dep[0] = 0; an[0] = 1ull; an[1] = 0ull;
    for (int n = 1; n < n_nodes; ++n) {
      if (par[n] < 0 || par[n] >= n) return fail(ctx, VADUSA_EINVAL, "node %d: parent %d must precede it", n, par[n]);
      dep[n] = dep[par[n]] + 1;
      an[2 * n] = an[2 * par[n]] | (n < 64 ? 1ull << n : 0ull);
      an[2 * n + 1] = an[2 * par[n] + 1] | (n >= 64 ? 1ull << (n - 64) : 0ull);
      if (dep[n] > VADUSA_MAX_DEPTH) return fail(ctx, VADUSA_EINVAL, "node %d: deeper than %d", n, VADUSA_MAX_DEPTH);
      if (!per_sequence) {
        if (dep[n] > ctx->cfg.n_draft_heads) return fail(ctx, VADUSA_EINVAL, "node %d: depth %d exceeds the number of draft heads", n, dep[n]);
        if (rnk[n] < 0 || rnk[n] >= ctx->cfg.draft_topk) return fail(ctx, VADUSA_EINVAL, "node %d: rank %d outside the draft top-k", n, rnk[n]);
      } else if (rnk[n] < 0) {
        return fail(ctx, VADUSA_EINVAL, "node %d: negative rank", n);
      }
      if (dep[n] < dep[n - 1]) return fail(ctx, VADUSA_EINVAL, "node %d: nodes must be ordered by depth", n);
      // (depth, rank path) order: within a depth, parents ascend, and siblings ascend by rank
      if (n > 1 && dep[n] == dep[n - 1]) {
        if (par[n] < par[n - 1] || (par[n] == par[n - 1] && rnk[n] <= rnk[n - 1]))
          return fail(ctx, VADUSA_EINVAL, "node %d: nodes of one depth must be in rank-path order", n);
      }
      max_rank = rnk[n] > max_rank ? rnk[n] : max_rank;
      max_depth = dep[n] > max_depth ? dep[n] : max_depth;
    }
  }
  const size_t n4 = (size_t)copies * n_nodes * sizeof(int32_t);
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.tree_parent, h_parent, n4, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.tree_rank, h_rank, n4, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.tree_depth, depth.data(), n4, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.tree_anc, anc.data(), (size_t)copies * n_nodes * 16, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  ctx->n_nodes = n_nodes;
  ctx->tree_per_seq = per_sequence ? 1 : 0;
  ctx->max_rank_used = max_rank;
  ctx->tree_max_depth = max_depth;
  ctx->have_draft = ctx->have_verify = false;
  if (ctx->batch > 0) return set_active(ctx, ctx->n_nodes);
  return VADUSA_OK;
}

vadusa_status vadusa_begin(vadusa_ctx* ctx, int32_t batch, const int32_t* block_table, const int32_t* h_ctx_len) {
  if (!ctx) return VADUSA_EINVAL;
  if (!ctx->wsp) return fail(ctx, VADUSA_ESTATE, "context is not initialised");
  if (batch < 1 || batch > ctx->cfg.max_batch) return fail(ctx, VADUSA_EINVAL, "batch must be in 1..max_batch");
  if (!block_table) return fail(ctx, VADUSA_EINVAL, "block_table is NULL");
  if (ctx->tree_per_seq) { ctx->n_nodes = 0; ctx->tree_per_seq = 0; }
  ctx->batch = batch;
  ctx->block_table = block_table;
  ctx->have_draft = ctx->have_verify = false;
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.scalars, 0, 256, ctx->stream));
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.f_sync, 0, 256, ctx->stream));
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.att_cnt, 0, 2 * kAsGrid * 4, ctx->stream));
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.gen_count, 0, batch * 4, ctx->stream));
  ctx->ctx_bound = 0;
  ctx->ctx_lo = 0;
  if (h_ctx_len) {
    for (int b = 0; b < batch; ++b) {
      if (h_ctx_len[b] < 0 || h_ctx_len[b] > (int64_t)ctx->cfg.max_blocks_per_seq * 64)
        return fail(ctx, VADUSA_EINVAL, "context length of sequence %d out of range", b);
      if (h_ctx_len[b] > ctx->ctx_bound) ctx->ctx_bound = h_ctx_len[b];
    }
    ctx->ctx_lo = ctx->ctx_bound;
    CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.ctx_len, h_ctx_len, batch * 4, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
  } else {
    CU(cudaMemsetAsync(ctx->wsp + ctx->ws.ctx_len, 0, batch * 4, ctx->stream));
  }
  return set_active(ctx, ctx->n_nodes);
}

vadusa_status vadusa_prefill(vadusa_ctx* ctx, const int32_t* h_tokens, const int32_t* h_len, int32_t stride) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (!h_tokens || !h_len || stride < 1) return fail(ctx, VADUSA_EINVAL, "prefill arguments are NULL or empty");
  vadusa_status s = DISPATCH(prefill<float>(ctx, h_tokens, h_len, stride), prefill<bf16>(ctx, h_tokens, h_len, stride));
  if (s) return s;

  ctx->have_draft = ctx->have_verify = false;
  return set_active(ctx, ctx->n_nodes);
}

vadusa_status vadusa_load_state(vadusa_ctx* ctx, const void* hstar, const float* logits_star) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (!hstar || !logits_star) return fail(ctx, VADUSA_EINVAL, "state pointers are NULL");
  const vadusa_config& c = ctx->cfg;
  CU(cudaMemcpyAsync(ctx->wsp + ctx->ws.hstar, hstar, (size_t)ctx->batch * c.d_model * esize(&c), cudaMemcpyDeviceToDevice, ctx->stream));
  CU(cudaMemcpy2DAsync(ctx->wsp + ctx->ws.logits_star, (size_t)vpad(&c) * 4, logits_star, (size_t)c.vocab * 4,
                       (size_t)c.vocab * 4, ctx->batch, cudaMemcpyDeviceToDevice, ctx->stream));
  return VADUSA_OK;
}

vadusa_status vadusa_draft(vadusa_ctx* ctx, const vadusa_sampling* sampling, int32_t* tree_tokens,
                           int32_t* draft_topk_out) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (ctx->n_nodes == 0) return fail(ctx, VADUSA_ESTATE, "no tree set");
  if (ctx->tree_per_seq && tree_tokens) return fail(ctx, VADUSA_EINVAL, "per-sequence topologies take their tokens from the override");
  SamplingDev sp;
  if (vadusa_status s = sampling_dev(ctx, sampling, &sp)) return s;
  const vadusa_config& c = ctx->cfg;
  const std::string key = KeyBuilder("draft").add(sp).add(tree_tokens).add(draft_topk_out).add(ctx->batch)
                              .add(ctx->n_nodes).add(ctx->tree_per_seq).add(ctx->block_table).k;
  vadusa_status s = run_graphed(ctx, key, [&]() -> vadusa_status {
    vadusa_status s = DISPATCH(draft<float>(ctx, sp), draft<bf16>(ctx, sp));
    if (s) return s;
    if (draft_topk_out)
      CU(cudaMemcpyAsync(draft_topk_out, ctx->wsp + ctx->ws.topk, (size_t)ctx->batch * c.n_draft_heads * c.draft_topk * 4,
                         cudaMemcpyDeviceToDevice, ctx->stream));
    if (tree_tokens) {
      // tokens of the tree without a model pass: the embed kernel computes them; run it alone
      const TreeView tv = tree_of(ctx, false);
      const int M = ctx->batch * tv.n_nodes;
      if (c.dtype == 1)
        tree_embed_kernel<bf16><<<M, 128, 0, ctx->stream>>>(
            tv, nullptr, wsptr<int32_t>(ctx, ctx->ws.root), wsptr<int32_t>(ctx, ctx->ws.topk), c.n_draft_heads, c.draft_topk,
            wsptr<int32_t>(ctx, ctx->ws.ctx_len), wsptr<int32_t>(ctx, ctx->ws.nvalid), as<bf16>(ctx->emb_audio),
            as<bf16>(ctx->emb_phon), as<bf16>(ctx->pos), c.vocab, c.n_phonemes, c.max_pos, c.d_model,
            wsptr<int32_t>(ctx, ctx->ws.tokens), wsptr<float>(ctx, ctx->ws.x), ctx->block_table, geom_of(ctx),
            (long long*)nullptr, (float2*)nullptr, err_word(ctx));
      else
        tree_embed_kernel<float><<<M, 128, 0, ctx->stream>>>(
            tv, nullptr, wsptr<int32_t>(ctx, ctx->ws.root), wsptr<int32_t>(ctx, ctx->ws.topk), c.n_draft_heads, c.draft_topk,
            wsptr<int32_t>(ctx, ctx->ws.ctx_len), wsptr<int32_t>(ctx, ctx->ws.nvalid), as<float>(ctx->emb_audio),
            as<float>(ctx->emb_phon), as<float>(ctx->pos), c.vocab, c.n_phonemes, c.max_pos, c.d_model,
            wsptr<int32_t>(ctx, ctx->ws.tokens), wsptr<float>(ctx, ctx->ws.x), ctx->block_table, geom_of(ctx),
            (long long*)nullptr, (float2*)nullptr, err_word(ctx));
      LAUNCH_CHECK();
      CU(cudaMemcpyAsync(tree_tokens, ctx->wsp + ctx->ws.tokens, (size_t)M * 4, cudaMemcpyDeviceToDevice, ctx->stream));
    }
    return VADUSA_OK;
  });
  if (s) return s;
  ctx->have_draft = true;
  return VADUSA_OK;
}

vadusa_status vadusa_verify_step(vadusa_ctx* ctx, const int32_t* tree_tokens_override, float* logits_out,
                                 void* attn_tap, void* hidden_out) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (ctx->n_nodes == 0) return fail(ctx, VADUSA_ESTATE, "no tree set");
  if (!tree_tokens_override && !ctx->have_draft) return fail(ctx, VADUSA_ESTATE, "verify without a draft or an override");
  if (!tree_tokens_override && ctx->tree_per_seq) return fail(ctx, VADUSA_ESTATE, "per-sequence topologies need a token override");
  const TreeView tv = tree_of(ctx, false);
  const vadusa_config& c = ctx->cfg;
  const int M = ctx->batch * tv.n_nodes;
  const std::string key = KeyBuilder("verify").add(tree_tokens_override).add(logits_out).add(attn_tap).add(hidden_out)
                              .add(ctx->batch).add(ctx->n_nodes).add(ctx->tree_per_seq).add(ctx->block_table)
                              .add(attention_splits(ctx, ctx->n_nodes)).add(ctx->fused_enabled).add(ctx->att_stream).k;
  vadusa_status s = run_graphed(ctx, key, [&]() -> vadusa_status {
    vadusa_status s = DISPATCH(forward<float>(ctx, tv, tree_tokens_override, reinterpret_cast<float*>(attn_tap)),
                               forward<bf16>(ctx, tv, tree_tokens_override, reinterpret_cast<bf16*>(attn_tap)));
    if (s) return s;
    if (logits_out)
      CU(cudaMemcpy2DAsync(logits_out, (size_t)c.vocab * 4, ctx->wsp + ctx->ws.logits, (size_t)vpad(&c) * 4,
                           (size_t)c.vocab * 4, M, cudaMemcpyDeviceToDevice, ctx->stream));
    if (hidden_out)
      CU(cudaMemcpyAsync(hidden_out, ctx->wsp + ctx->ws.hfinal, (size_t)M * c.d_model * esize(&c), cudaMemcpyDeviceToDevice, ctx->stream));
    return VADUSA_OK;
  });
  if (s) return s;
  ctx->have_verify = true;
  return VADUSA_OK;
}

vadusa_status vadusa_accept_and_commit(vadusa_ctx* ctx, const vadusa_sampling* sampling, const int32_t* forced_best_node,
                                       int32_t* accept_len, int32_t* path_nodes, int32_t* path_tokens,
                                       int64_t* kv_slots, uint64_t* edge_bits, int32_t* next_root) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (!ctx->have_verify) return fail(ctx, VADUSA_ESTATE, "accept without a verify step");
  SamplingDev sp;
  if (vadusa_status s = sampling_dev(ctx, sampling, &sp)) return s;
  AcceptOut out{accept_len, path_nodes, path_tokens, reinterpret_cast<long long*>(kv_slots),
                reinterpret_cast<unsigned long long*>(edge_bits), ctx->cfg.max_tree_nodes > 64 ? 2 : 1, next_root};
  const std::string key = KeyBuilder("accept").add(sp).add(forced_best_node).add(out).add(ctx->batch).add(ctx->n_nodes)
                              .add(ctx->tree_per_seq).add(ctx->block_table).k;
  vadusa_status s = run_graphed(ctx, key, [&]() -> vadusa_status {
    return DISPATCH(accept_commit<float>(ctx, sp, forced_best_node, out, nullptr, 0, 0),
                    accept_commit<bf16>(ctx, sp, forced_best_node, out, nullptr, 0, 0));
  });
  if (s) return s;
  ctx->ctx_bound += ctx->tree_max_depth + 1;
  ctx->ctx_lo += 1;
  ctx->have_verify = ctx->have_draft = false;
  return VADUSA_OK;
}

vadusa_status vadusa_generate(vadusa_ctx* ctx, const vadusa_sampling* sampling, int32_t max_new_tokens,
                              int32_t max_iters, int32_t* out_tokens, int32_t* out_len, vadusa_stats* h_stats) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (ctx->n_nodes == 0 || ctx->tree_per_seq) return fail(ctx, VADUSA_ESTATE, "generate needs a shared tree template");
  if (max_new_tokens < 1) return fail(ctx, VADUSA_EINVAL, "max_new_tokens must be positive");
  SamplingDev sp;
  if (vadusa_status s = sampling_dev(ctx, sampling, &sp)) return s;
  const int64_t launches0 = ctx->launches;
  const int limit = max_iters > 0 ? max_iters : max_new_tokens;
  const TreeView tv = tree_of(ctx, false);
  AcceptOut none{nullptr, nullptr, nullptr, nullptr, nullptr, 1, nullptr};
  CU(cudaMemsetAsync(ctx->wsp + ctx->ws.gen_count, 0, ctx->batch * 4, ctx->stream));
  CU(cudaMemsetAsync(done_word(ctx), 0, 4, ctx->stream));
  if (vadusa_status s = set_active(ctx, ctx->n_nodes)) return s;
  ctx->h_pinned[0] = 0;
  bool poll_pending = false;
  int iters = 0;
  CU(cudaEventRecord(ctx->ev0, ctx->stream));
  for (; iters < limit; ++iters) {
    if (poll_pending && cudaEventQuery(ctx->ev_poll) == cudaSuccess) {
      poll_pending = false;
      if (ctx->h_pinned[0] >= ctx->batch) break;
    }
    // stay at most sixteen iterations ahead of the device: when the next poll is due and the last one has not come
    // back, wait for it (iterations enqueued behind the end of the last sequence find nothing to do, but cost time)
    if (poll_pending && (iters & 7) == 7) {
      CU(cudaEventSynchronize(ctx->ev_poll));
      poll_pending = false;
      if (ctx->h_pinned[0] >= ctx->batch) break;
    }
    const std::string iter_key = KeyBuilder("iteration").add(sp).add(out_tokens).add(max_new_tokens).add(ctx->batch)
                                     .add(ctx->n_nodes).add(ctx->block_table).add(attention_splits(ctx, ctx->n_nodes)).add(ctx->fused_enabled).add(ctx->att_stream).k;
    vadusa_status s = run_graphed(ctx, iter_key, [&]() -> vadusa_status {
      vadusa_status s = DISPATCH(draft<float>(ctx, sp), draft<bf16>(ctx, sp));
      if (s) return s;
      s = DISPATCH(forward<float>(ctx, tv, nullptr, nullptr), forward<bf16>(ctx, tv, nullptr, nullptr));
      if (s) return s;
      return DISPATCH(accept_commit<float>(ctx, sp, nullptr, none, out_tokens, max_new_tokens, max_new_tokens),
                      accept_commit<bf16>(ctx, sp, nullptr, none, out_tokens, max_new_tokens, max_new_tokens));
    });
    if (s) return s;
    ctx->ctx_bound += ctx->tree_max_depth + 1;
    ctx->ctx_lo += 1;
    if (!poll_pending && (iters & 7) == 7) {
      CU(cudaMemcpyAsync(ctx->h_pinned, done_word(ctx), 4, cudaMemcpyDeviceToHost, ctx->stream));
      CU(cudaEventRecord(ctx->ev_poll, ctx->stream));
      poll_pending = true;
    }
  }
  CU(cudaEventRecord(ctx->ev1, ctx->stream));
  // lengths: min(gen_count, max_new_tokens) — computed on the host after the final sync
  std::vector<int32_t> gen(ctx->batch);
  CU(cudaMemcpyAsync(gen.data(), ctx->wsp + ctx->ws.gen_count, ctx->batch * 4, cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  int64_t total = 0;
  for (int b = 0; b < ctx->batch; ++b) { total += gen[b]; gen[b] = gen[b] > max_new_tokens ? max_new_tokens : gen[b]; }
  if (out_len) CU(cudaMemcpyAsync(out_len, gen.data(), ctx->batch * 4, cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  if (h_stats) {
    float ms = 0.f;
    CU(cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
    h_stats->iterations = iters;
    h_stats->tokens_generated = total;
    h_stats->elapsed_ms = ms;
    h_stats->kernel_launches = ctx->launches - launches0;
  }
  ctx->have_draft = ctx->have_verify = false;
  return device_errors(ctx);
}

vadusa_status vadusa_generate_host(vadusa_ctx* ctx, const vadusa_sampling* sampling, int32_t batch,
                                   const int32_t* block_table, const int32_t* h_tokens, const int32_t* h_len,
                                   int32_t stride, int32_t max_new_tokens, int32_t* h_out_tokens,
                                   int32_t* h_out_len, vadusa_stats* h_stats) {
  if (!ctx) return VADUSA_EINVAL;
  if (!h_out_tokens || !h_out_len) return fail(ctx, VADUSA_EINVAL, "output pointers are NULL");
  if (max_new_tokens < 1 || max_new_tokens > kGenHostCap)
    return fail(ctx, VADUSA_EINVAL, "vadusa_generate_host: max_new_tokens must be in 1..%d", kGenHostCap);
  vadusa_status s = vadusa_begin(ctx, batch, block_table, nullptr);
  if (s) return s;
  s = vadusa_prefill(ctx, h_tokens, h_len, stride);
  if (s) return s;
  int32_t* d_out = wsptr<int32_t>(ctx, ctx->ws.gen_out);
  int32_t* d_len = wsptr<int32_t>(ctx, ctx->ws.gen_len);
  s = vadusa_generate(ctx, sampling, max_new_tokens, 0, d_out, d_len, h_stats);
  if (s == VADUSA_OK) {
    cudaMemcpyAsync(h_out_tokens, d_out, (size_t)batch * max_new_tokens * 4, cudaMemcpyDeviceToHost, ctx->stream);
    cudaMemcpyAsync(h_out_len, d_len, (size_t)batch * 4, cudaMemcpyDeviceToHost, ctx->stream);
  }
  CU(cudaStreamSynchronize(ctx->stream));
  return s;
}

vadusa_status vadusa_get_lengths(vadusa_ctx* ctx, int32_t* h_ctx_len) {
  if (vadusa_status s = need_batch(ctx)) return s;
  if (!h_ctx_len) return fail(ctx, VADUSA_EINVAL, "h_ctx_len is NULL");
  CU(cudaMemcpyAsync(h_ctx_len, ctx->wsp + ctx->ws.ctx_len, ctx->batch * 4, cudaMemcpyDeviceToHost, ctx->stream));
  if (vadusa_status s = device_errors(ctx)) return s;       // (synchronises)
  long long longest = 0;
  for (int b = 0; b < ctx->batch; ++b) longest = h_ctx_len[b] > longest ? h_ctx_len[b] : longest;
  ctx->ctx_lo = ctx->ctx_bound = longest;                   // both estimates are exact again
  return VADUSA_OK;
}

vadusa_status vadusa_check(vadusa_ctx* ctx) {
  if (!ctx || !ctx->wsp) return VADUSA_EINVAL;
  return device_errors(ctx);
}

vadusa_status vadusa_set_logit_bias(vadusa_ctx* ctx, const float* bias, int32_t ld) {
  if (!ctx) return VADUSA_EINVAL;
  if (!ctx->wsp) return fail(ctx, VADUSA_ESTATE, "context is not initialised");
  if (bias && ld < ctx->cfg.vocab) return fail(ctx, VADUSA_EINVAL, "bias rows must hold at least vocab entries");
  ctx->logit_bias = bias;
  ctx->logit_bias_ld = bias ? ld : 0;
  return VADUSA_OK;
}

vadusa_status vadusa_accept_stats(vadusa_ctx* ctx, int64_t* h_tested, int64_t* h_accepted, int32_t reset) {
  if (!ctx) return VADUSA_EINVAL;
  if (!ctx->wsp) return fail(ctx, VADUSA_ESTATE, "context is not initialised");
  if (!h_tested || !h_accepted) return fail(ctx, VADUSA_EINVAL, "statistics arrays are NULL");
  const size_t n = (size_t)kStatDepth * kStatTopk;
  static_assert(sizeof(int64_t) == sizeof(unsigned long long), "counter width");
  CU(cudaMemcpyAsync(h_tested, ctx->wsp + ctx->ws.acc_stats, n * 8, cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaMemcpyAsync(h_accepted, ctx->wsp + ctx->ws.acc_stats + n * 8, n * 8, cudaMemcpyDeviceToHost, ctx->stream));
  if (reset) CU(cudaMemsetAsync(ctx->wsp + ctx->ws.acc_stats, 0, 2 * n * 8, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return VADUSA_OK;
}

vadusa_status vadusa_build_sparse_tree(const double* h_prob, int32_t depth, int32_t topk, int32_t n_nodes,
                                       int32_t* h_parent, int32_t* h_rank, double* h_expected_len) {
  if (!h_prob || !h_parent || !h_rank) return VADUSA_EINVAL;
  if (depth < 1 || depth > VADUSA_MAX_DEPTH || topk < 1 || topk > VADUSA_MAX_DRAFT_TOPK) return VADUSA_EINVAL;
  if (n_nodes < 1 || n_nodes > VADUSA_MAX_TREE_NODES) return VADUSA_EINVAL;
  struct Node { std::vector<int> path; double p; };
  auto before = [](const Node& a, const Node& b) {       // higher probability, then shallower, then smaller path
    if (a.p != b.p) return a.p > b.p;
    if (a.path.size() != b.path.size()) return a.path.size() < b.path.size();
    return a.path < b.path;
  };
  std::vector<Node> tree(1, Node{{}, 1.0}), frontier;
  auto grow = [&](const Node& parent) {
    if ((int)parent.path.size() == depth) return;
    for (int r = 0; r < topk; ++r) {
      Node c{parent.path, parent.p * h_prob[(size_t)parent.path.size() * topk + r]};
      c.path.push_back(r);
      frontier.push_back(c);
    }
  };
  grow(tree[0]);
  double expected = 1.0;
  while ((int)tree.size() < n_nodes) {
    if (frontier.empty()) return VADUSA_EINVAL;
    size_t best = 0;
    for (size_t i = 1; i < frontier.size(); ++i)
      if (before(frontier[i], frontier[best])) best = i;
    const Node pick = frontier[best];
    frontier.erase(frontier.begin() + (long)best);
    expected += pick.p;
    tree.push_back(pick);
    grow(pick);
  }
  std::sort(tree.begin(), tree.end(), [](const Node& a, const Node& b) {
    return a.path.size() != b.path.size() ? a.path.size() < b.path.size() : a.path < b.path;
  });
  std::map<std::vector<int>, int> index;
  for (int i = 0; i < n_nodes; ++i) index[tree[i].path] = i;
  for (int i = 0; i < n_nodes; ++i) {
    if (tree[i].path.empty()) { h_parent[i] = -1; h_rank[i] = 0; continue; }
    std::vector<int> up(tree[i].path.begin(), tree[i].path.end() - 1);
    h_parent[i] = index[up];
    h_rank[i] = tree[i].path.back();
  }
  if (h_expected_len) *h_expected_len = expected;
  return VADUSA_OK;
}

int64_t vadusa_fit_state_bytes(const vadusa_config* cfg, int32_t max_tokens) {
  if (check_config(cfg) || max_tokens < 1) return -1;
  return fit_layout(cfg, max_tokens).total;
}

vadusa_status vadusa_fit_begin(vadusa_ctx* ctx, void* state, int64_t state_bytes, int32_t max_tokens, float lambda,
                               float learning_rate, int32_t warmup_steps) {
  if (!ctx) return VADUSA_EINVAL;
  if (!ctx->wsp) return fail(ctx, VADUSA_ESTATE, "context is not initialised");
  if (!state || max_tokens < 1 || ((uintptr_t)state & 255)) return fail(ctx, VADUSA_EINVAL, "fit state is NULL, unaligned or sized for no token");
  if (!(lambda > 0.f && lambda <= 1.f) || !(learning_rate > 0.f) || warmup_steps < 0) return fail(ctx, VADUSA_EINVAL, "lambda must be in (0, 1], the learning rate positive");
  const FitLayout f = fit_layout(&ctx->cfg, max_tokens);
  if (state_bytes < f.total) return fail(ctx, VADUSA_ENOMEM, "fit state has %lld bytes, %lld needed", (long long)state_bytes, (long long)f.total);
  if (ctx->cfg.n_draft_heads > 1 && ctx->dw_stride != (long long)ctx->cfg.d_model * ctx->cfg.d_model * esize(&ctx->cfg))
    return fail(ctx, VADUSA_EINVAL, "draft matrices are not contiguous");
  ctx->fit = reinterpret_cast<char*>(state);
  ctx->fit_tokens = max_tokens; ctx->fit_step = 0; ctx->fit_warmup = warmup_steps;
  ctx->fit_lambda = lambda; ctx->fit_lr = learning_rate;
  return DISPATCH(fit_begin<float>(ctx, f), fit_begin<bf16>(ctx, f));
}

vadusa_status vadusa_fit_step(vadusa_ctx* ctx, const void* hidden, const int32_t* targets, int32_t n_tokens, float* loss_out) {
  if (!ctx) return VADUSA_EINVAL;
  if (!ctx->fit) return fail(ctx, VADUSA_ESTATE, "vadusa_fit_begin has not been called");
  if (!hidden || !targets || n_tokens < 1 || n_tokens > ctx->fit_tokens) return fail(ctx, VADUSA_EINVAL, "fit step: NULL input or token count out of range");
  const FitLayout f = fit_layout(&ctx->cfg, ctx->fit_tokens);
  ctx->have_draft = false;
  return DISPATCH(fit_step<float>(ctx, f, reinterpret_cast<const float*>(hidden), targets, n_tokens, loss_out),
                  fit_step<bf16>(ctx, f, reinterpret_cast<const bf16*>(hidden), targets, n_tokens, loss_out));
}

vadusa_status vadusa_fit_end(vadusa_ctx* ctx) {
  if (!ctx) return VADUSA_EINVAL;
  ctx->fit = nullptr;
  return VADUSA_OK;
}

vadusa_status vadusa_set_prefill_tap(vadusa_ctx* ctx, void* hidden_out, int32_t stride) {
  if (!ctx) return VADUSA_EINVAL;
  if (hidden_out && stride < 1) return fail(ctx, VADUSA_EINVAL, "prefill tap: stride must be positive");
  ctx->pf_tap = hidden_out;
  ctx->pf_tap_stride = hidden_out ? stride : 0;
  return VADUSA_OK;
}

int64_t vadusa_kernel_launches(const vadusa_ctx* ctx) { return ctx ? ctx->launches : 0; }

int32_t vadusa_fused_pass_clusters(const vadusa_ctx* ctx) { return ctx ? ctx->fused_clusters : -1; }

vadusa_status vadusa_set_attention_stream(vadusa_ctx* ctx, int32_t enable) {
  if (!ctx) return VADUSA_EINVAL;
  if (enable != 0 && enable != 1) return fail(ctx, VADUSA_EINVAL, "enable must be 0 or 1");
  ctx->att_stream = enable;
  return VADUSA_OK;
}

vadusa_status vadusa_set_fused_pass(vadusa_ctx* ctx, int32_t enable) {
  if (!ctx) return VADUSA_EINVAL;
  if (enable != 0 && enable != 1 && enable != 6 && enable != 8) return fail(ctx, VADUSA_EINVAL, "enable must be 0, 1, 6 or 8");
  ctx->fused_enabled = enable;
  return VADUSA_OK;
}

vadusa_status vadusa_profile_begin(vadusa_ctx* ctx) {
  if (!ctx || !ctx->wsp) return VADUSA_EINVAL;
  for (auto& r : ctx->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  ctx->prof.clear();
  ctx->prof_on = true;
  ctx->prof_pending = false;
  return VADUSA_OK;
}

vadusa_status vadusa_profile_end(vadusa_ctx* ctx, vadusa_kernel_time* h_out, int32_t capacity, int32_t* h_count) {
  if (!ctx || !ctx->wsp) return VADUSA_EINVAL;
  if (!h_out || !h_count || capacity < K_NCLASS) return fail(ctx, VADUSA_EINVAL, "profile output needs room for %d entries", (int)K_NCLASS);
  ctx->prof_on = false;
  CU(cudaStreamSynchronize(ctx->stream));
  double total[K_NCLASS] = {0};
  int64_t count[K_NCLASS] = {0};
  for (auto& r : ctx->prof) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) { total[r.cls] += ms; count[r.cls]++; }
    cudaEventDestroy(r.a); cudaEventDestroy(r.b);
  }
  ctx->prof.clear();
  int n = 0;
  for (int k = 0; k < K_NCLASS; ++k) {
    if (!count[k]) continue;
    memset(&h_out[n], 0, sizeof(h_out[n]));
    snprintf(h_out[n].name, sizeof(h_out[n].name), "%s", kClassName[k]);
    h_out[n].launches = count[k];
    h_out[n].total_ms = total[k];
    ++n;
  }
  *h_count = n;
  return VADUSA_OK;
}

}  // extern "C"
