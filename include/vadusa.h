/*
 * vadusa.h — C ABI of libvadusa: the tree draft-and-verify step of VADUSA
 * (MEDUSA-style speculative decoding with a tolerance rule for a VALL-E-style
 * decoder-only speech-token language model) on NVIDIA B200 (sm_100a).
 *
 * Conventions
 *  - Every call returns a vadusa_status; no C++ exception crosses this boundary.
 *  - Pointers are DEVICE pointers unless the parameter name starts with h_ (host).
 *    Any output pointer may be NULL, which means "do not write it".
 *  - The caller owns every buffer it passes (weights, KV pool, workspace, block
 *    table, inputs, outputs) and keeps it alive until vadusa_destroy.  The
 *    library owns only the opaque vadusa_ctx (host memory, two CUDA events and
 *    a few pinned host words).
 *  - All device work is enqueued on the stream given in the configuration, in
 *    call order; calls do not synchronise unless they say so.
 *  - Errors found on the host make the call return at once with a message in
 *    vadusa_last_error.  Errors found on the device (capacity exhausted, a
 *    bounded wait that expired) set bits in a device error word; they surface
 *    as the return value of the next call that synchronises
 *    (vadusa_get_lengths, vadusa_generate, vadusa_check).
 *  - There is no CPU path: if no sm_100 device is present vadusa_init fails
 *    with VADUSA_ECUDA.
 *
 * Model (paper Sec. III-A.1; details the paper leaves to VALL-E are fixed here):
 *  a pre-LayerNorm decoder-only transformer with learned absolute positions,
 *  multi-head attention (every head has its own K/V), ReLU feed-forward, biases
 *  on all projections except the vocabulary heads, LayerNorm with affine
 *  parameters, one running position index over [phonemes ; prompt ; generated].
 *  Phoneme tokens use their own embedding table; on this interface a phoneme id
 *  p is written as the token id vocab + p.
 *  Draft head i (i = 1..n_draft_heads) is z = h + SiLU(W_i h + b_i), then its own
 *  vocabulary projection U_i z (Sec. II-A, III-A.1); h is the final-LayerNorm
 *  output at the last committed token.
 *
 * Numeric types: dtype 0 keeps weights, K/V and activations in fp32 (plain
 *  fp32 FMA arithmetic).  dtype 1 keeps matrices, embeddings, K/V and the
 *  activations that feed a matrix product in bf16 (rounded to nearest even
 *  where produced: LayerNorm outputs, q/k/v, attention output, feed-forward
 *  hidden layer, final hidden state, draft residual block output) and
 *  accumulates in fp32; the residual stream, softmax weights and statistics,
 *  logits and sampling keys are fp32 (the softmax weights enter the P.V product
 *  with at least 16 significant bits).
 */
#ifndef VADUSA_H
#define VADUSA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VADUSA_ABI_VERSION 2u
#define VADUSA_MAX_TREE_NODES 128  /* two 64-bit ancestor words per node (the paper's 64-, 96- and 128-node trees) */
#define VADUSA_MAX_DRAFT_TOPK 16
#define VADUSA_MAX_DEPTH 15        /* a root path has at most 16 nodes */

typedef enum {
  VADUSA_OK = 0,
  VADUSA_EINVAL = 1,     /* bad argument or configuration */
  VADUSA_ENOMEM = 2,     /* caller's workspace / KV pool / weight blob too small */
  VADUSA_ECUDA = 3,      /* a CUDA runtime or driver call failed */
  VADUSA_ECAPACITY = 4,  /* a sequence ran out of KV blocks, positions or output room */
  VADUSA_ESTATE = 5,     /* call order (e.g. verify before a tree was set) */
  VADUSA_ETIMEOUT = 6    /* a bounded device-side wait expired */
} vadusa_status;

typedef struct vadusa_ctx vadusa_ctx;

typedef struct {
  uint32_t struct_size;        /* sizeof(vadusa_config) */
  uint32_t abi_version;        /* VADUSA_ABI_VERSION */
  int32_t n_layers, d_model, n_heads, d_ffn;
  int32_t vocab;               /* speech-token ids, the last one (vocab-1) is EOS; 2..24576 */
  int32_t n_phonemes;
  int32_t max_pos;             /* rows of the position table */
  int32_t dtype;               /* 0 fp32, 1 bf16 */
  int32_t n_draft_heads;       /* <= VADUSA_MAX_DEPTH */
  int32_t draft_topk;          /* candidates kept per draft head, <= VADUSA_MAX_DRAFT_TOPK */
  int32_t max_batch;
  int32_t max_tree_nodes;      /* <= VADUSA_MAX_TREE_NODES */
  int32_t kv_block;            /* tokens per KV block; must be 64 */
  int32_t max_blocks_per_seq;  /* row length of the block table */
  int32_t prefill_rows;        /* chunks of max_tree_nodes prefix tokens that one prefill pass scores together
                                  (sizes the activation buffers with max(max_batch, prefill_rows) rows of
                                  max_tree_nodes tokens); 0 = max_batch; <= 4096 */
  int32_t reserved0;           /* must be 0 */
  int64_t kv_num_blocks;       /* blocks per layer in the pool */
  float ln_eps;
  int32_t device;              /* CUDA device ordinal */
  void *kv_pool;               /* [n_layers][kv_num_blocks][2 (K,V)][n_heads][kv_block][head_dim] of dtype */
  int64_t kv_pool_bytes;
  void *workspace;             /* >= vadusa_workspace_bytes(cfg) bytes, 256-byte aligned */
  int64_t workspace_bytes;
  void *stream;                /* cudaStream_t; NULL = the legacy default stream */
} vadusa_config;

/* The weight blob: all tensors back to back in device memory, in the order and at
 * the offsets reported by vadusa_weight_info.  Matrices are row-major
 * [out_features][in_features] in the model dtype; the vocabulary matrices ("lm",
 * "draft<i>.u") have their rows padded with zeros to a multiple of 128; vectors
 * (biases, LayerNorm gains and offsets) are fp32. */
typedef struct { const void *blob; int64_t nbytes; } vadusa_weights;

typedef struct {
  char name[32];       /* "emb_audio", "emb_phon", "pos", "l<k>.ln1_g", "l<k>.wqkv", ..., "lnf_g", "lm", "draft<i>.w" ... */
  int64_t offset;      /* byte offset in the blob, a multiple of 256 */
  int64_t nbytes;
  int32_t rows, cols;  /* logical shape (cols = 1 for vectors) */
  int32_t rows_padded; /* rows as stored */
  int32_t is_matrix;   /* 1: stored in the model dtype; 0: fp32 vector */
} vadusa_tensor_info;

/* Sampling of the base head and the acceptance rule (Algorithm 1, Sec. II-C).
 * At every scored node the base head "samples tau times"; a child candidate is
 * accepted if it is one of those samples.  The tau samples are drawn without
 * replacement from the top-p nucleus of softmax(logits / temperature) by
 * perturbing logits/temperature with Gumbel noise and taking the tau largest
 * keys; the first of them is the ordinary single sample.  The noise is a pure
 * function of (seed, sequence index, absolute position of the predicted token,
 * token id): 23 bits of a three-stage splitmix64 hash give u = (x + 1/2) / 2^23,
 * g = -log(-log(u)) in fp32, key = logit * (1/temperature) + g in fp32.  Ties
 * go to the lower token id.  temperature 0 means greedy: keys are the logits
 * and top_p is ignored.  top_p >= 1 switches the nucleus off. */
typedef struct {
  int32_t tau;           /* tolerance, >= 1 */
  float temperature;     /* 0 = greedy */
  float top_p;
  int32_t eos_masked;    /* 1: the EOS logit counts as -inf everywhere (base and draft heads); generation ends by
                            length.  0: EOS can be drawn and drafted; a sequence ends (becomes inactive) in the
                            iteration that commits EOS, and the tokens behind EOS on the accepted path are
                            dropped (tolerance 1 then stops exactly where plain decoding stops, Sec. II-A) */
  int32_t accept_rule;   /* 0: Algorithm 1 as above; 1: membership in the plain top-tau of the
                            unperturbed logits (the root is still sampled with noise) */
  uint64_t seed;
} vadusa_sampling;

typedef struct {
  int64_t iterations;        /* draft-and-verify iterations run */
  int64_t tokens_generated;  /* over all sequences */
  double elapsed_ms;         /* device time of the loop (CUDA events) */
  int64_t kernel_launches;   /* kernels of this library enqueued by the call */
} vadusa_stats;

/* ---- sizing and layout (host only, no GPU needed) ------------------------------ */
int64_t vadusa_workspace_bytes(const vadusa_config *cfg);       /* < 0 on a bad configuration */
int64_t vadusa_weights_bytes(const vadusa_config *cfg);
int64_t vadusa_kv_pool_bytes(const vadusa_config *cfg);
int32_t vadusa_weight_count(const vadusa_config *cfg);
vadusa_status vadusa_weight_info(const vadusa_config *cfg, int32_t index, vadusa_tensor_info *h_out);

/* ---- life cycle ------------------------------------------------------------------ */
/* Binds a context to one model: the decoder-only speech-token model of Sec. III-A.1 (12 layers, 16 heads,
 * d 1024, feed-forward 4096 in the paper; any shape the configuration checks allow) and its draft heads
 * (Sec. II-A: one residual Linear+SiLU block and one vocabulary matrix per head).
 * Validates the configuration, records the pointers, clears the state area of the
 * workspace.  Synchronises the stream once.  Makes cfg->device the calling thread's current
 * CUDA device; every later call on the context must be made with that device current.  A
 * context is not thread-safe: one thread at a time. */
vadusa_status vadusa_init(const vadusa_weights *weights, const vadusa_config *cfg, vadusa_ctx **h_out);
vadusa_status vadusa_destroy(vadusa_ctx *ctx);
const char *vadusa_last_error(const vadusa_ctx *ctx);   /* NUL-terminated, owned by the context */

/* The static candidate tree (Sec. II-A, II-D): node 0 is the root (the base head's
 * own next token); node n >= 1 has parent h_parent[n] < n and holds candidate
 * number h_rank[n] (0 = best) of draft head depth(n).  Nodes must come in
 * (depth, rank path) order so that, among equally deep nodes, a smaller index is
 * a more-left branch.  per_sequence = 0: one template [n_nodes] for all sequences.
 * per_sequence = 1: arrays are [batch][n_nodes], one topology per sequence
 * (call after vadusa_begin).  Host arrays; copied. */
vadusa_status vadusa_set_tree(vadusa_ctx *ctx, int32_t n_nodes, const int32_t *h_parent,
                              const int32_t *h_rank, int32_t per_sequence);

/* Starts a batch of independent utterances (Sec. II-A treats one; nothing is exchanged between sequences,
 * each has its own context, tree scores and acceptance).  block_table: device int32 [batch][max_blocks_per_seq], the KV
 * blocks of every sequence in logical order; it must cover every position the
 * sequence can reach plus max_tree_nodes (tree nodes are scored in place behind the
 * context).  h_ctx_len: host int32 [batch], tokens already present in the cache
 * (NULL = all zero). */
vadusa_status vadusa_begin(vadusa_ctx *ctx, int32_t batch, const int32_t *block_table,
                           const int32_t *h_ctx_len);

/* Feeds the prefix [phonemes ; prompt speech tokens] of every sequence through the
 * model (paper Fig. 1a) behind whatever the cache already holds.  The prefixes are cut
 * into chunks of max_tree_nodes tokens; a chunk is scored as a chain-shaped tree (all
 * nodes accepted) whose context is everything before it, and up to max(max_batch,
 * prefill_rows) chunks -- of one sequence or of several -- go through the model in one
 * pass: every chunk's K/V rows are in the cache before the pass's attention reads
 * them, so later chunks of a sequence see the earlier ones of the same pass.
 * h_tokens: host int32 [batch][stride], phoneme p written as vocab + p; h_len: host
 * int32 [batch].  Leaves the hidden state and base-head logits of the last prefix
 * token as the start of decoding.  Synchronises the stream. */
vadusa_status vadusa_prefill(vadusa_ctx *ctx, const int32_t *h_tokens, const int32_t *h_len, int32_t stride);

/* Microbenchmark / test entry: sets the carried state directly.  hstar: [batch][d_model]
 * in the model dtype; logits_star: fp32 [batch][vocab]. */
vadusa_status vadusa_load_state(vadusa_ctx *ctx, const void *hstar, const float *logits_star);

/* ---- the hot path ------------------------------------------------------------------ */
/* Draft (Sec. II-A): root = the base head's sample for the next position, from the
 * carried logits; every draft head's top-k at the carried hidden state; tokens
 * scattered into the tree.  tree_tokens: int32 [batch][n_nodes] out.
 * draft_topk_out: int32 [batch][n_draft_heads][draft_topk] out. */
vadusa_status vadusa_draft(vadusa_ctx *ctx, const vadusa_sampling *sampling, int32_t *tree_tokens,
                           int32_t *draft_topk_out);

/* Verify (Sec. II-A "tree attention", Alg. 1 line 1): one forward pass of the base
 * model over all tree nodes; node n sits at position ctx_len + depth(n), attends to
 * the whole cached context and to its ancestors and itself.  Its K/V rows are
 * written behind the context (slot ctx_len + n).  tree_tokens_override: int32
 * [batch][n_nodes] replaces the drafted tokens (test hook; NULL = use the draft).
 * logits_out: fp32 [batch][n_nodes][vocab]; attn_tap: [n_layers][batch][n_nodes][d_model]
 * in the model dtype (attention output before the output projection);
 * hidden_out: [batch][n_nodes][d_model] final-LayerNorm output in the model dtype. */
vadusa_status vadusa_verify_step(vadusa_ctx *ctx, const int32_t *tree_tokens_override,
                                 float *logits_out, void *attn_tap, void *hidden_out);

/* Accept and commit (Alg. 1 lines 2-15, Sec. II-C): per edge, is the child token among
 * the tau draws at its parent; a node is accepted if its whole root path is; the
 * deepest accepted node wins, the smallest index among equally deep ones; the K/V
 * rows of its path move to slots ctx_len .. ctx_len + accept_len - 1, its hidden state
 * and logits become the carried state, ctx_len grows by accept_len.
 * forced_best_node: int32 [batch] overrides the winner (test hook; -1 entries keep the rule).
 * accept_len int32 [batch]; path_nodes, path_tokens int32 [batch][VADUSA_MAX_DEPTH+1]
 * (entries beyond accept_len are -1); kv_slots int64 [batch][VADUSA_MAX_DEPTH+1]:
 * block * kv_block + offset of every committed token; edge_bits uint64 [batch][W], W = 1 if
 * the configuration's max_tree_nodes <= 64, else 2: bit n (of word n / 64) set iff edge
 * parent(n)->n was tested and accepted (bit 0 always set); next_root int32 [batch]:
 * the base head's sample for the position after the winner. */
vadusa_status vadusa_accept_and_commit(vadusa_ctx *ctx, const vadusa_sampling *sampling,
                                       const int32_t *forced_best_node, int32_t *accept_len,
                                       int32_t *path_nodes, int32_t *path_tokens, int64_t *kv_slots,
                                       uint64_t *edge_bits, int32_t *next_root);

/* The decoding loop of Sec. II-A (Fig. 1b-c): draft heads propose, the base model scores the candidate tree in
 * one pass, Algorithm 1 keeps the longest accepted path, and the base head's distribution at the last accepted
 * token starts the next iteration.
 * Runs draft -> verify -> accept+commit until every sequence has max_new_tokens tokens
 * (or max_iters iterations, if > 0).  out_tokens: int32 [batch][max_new_tokens]
 * (a sequence's surplus tokens of its last iteration are dropped); out_len: int32
 * [batch].  Synchronises; returns device-side errors.  h_stats may be NULL. */
vadusa_status vadusa_generate(vadusa_ctx *ctx, const vadusa_sampling *sampling, int32_t max_new_tokens,
                              int32_t max_iters, int32_t *out_tokens, int32_t *out_len,
                              vadusa_stats *h_stats);

/* The same from host memory to host memory (what an application calls): begin,
 * prefill from h_tokens, generate, copy the tokens back.  block_table is a device
 * pointer as in vadusa_begin; all other buffers are host memory.  Synchronises. */
vadusa_status vadusa_generate_host(vadusa_ctx *ctx, const vadusa_sampling *sampling, int32_t batch,
                                   const int32_t *block_table, const int32_t *h_tokens,
                                   const int32_t *h_len, int32_t stride, int32_t max_new_tokens,
                                   int32_t *h_out_tokens, int32_t *h_out_len, vadusa_stats *h_stats);

/* ---- state ---------------------------------------------------------------------- */
/* Tokens in each sequence's cache: prefix plus what the iterations so far have committed (Sec. II-A: an
 * iteration commits between 1 and n_draft_heads + 1 tokens, so the length is the only way to know how far a
 * sequence has come).  h_ctx_len: host int32 [batch].  Synchronises; returns device-side errors. */
vadusa_status vadusa_get_lengths(vadusa_ctx *ctx, int32_t *h_ctx_len);
vadusa_status vadusa_check(vadusa_ctx *ctx);                            /* synchronises; device error word */
int64_t vadusa_kernel_launches(const vadusa_ctx *ctx);                  /* total kernels enqueued so far */

/* Tree attention of a batch (Sec. II-A) runs with one thread block per (head, sequence), the sequences visited
 * longest first.  For bf16 models with head_dim 64, at most 64 tree nodes, at most 512 sequences and enough
 * (sequence, head) pairs to fill the device, enable = 1 selects a persistent kernel instead in which every thread
 * block takes an equal share of the stream of K/V pages of all sequences, whatever their lengths; a pair whose
 * pages fall to several blocks is merged by the block that finishes last, in the order of the pages.  Both
 * compute the same attention with the same rounding points per page.  enable = 0 is the default: it is the faster one on the
 * devices measured so far.  Host-side switch: takes effect with the next call. */
vadusa_status vadusa_set_attention_stream(vadusa_ctx *ctx, int32_t enable);

/* A verify pass over ONE sequence of at most 64 tree nodes (the batch-1 step of Sec. II-A: one tree per
 * iteration) can run, for bf16 models with head_dim 64 and 8 or 16 heads, as a single persistent kernel that
 * keeps the whole grid resident (one thread-block cluster per head), lets weights and context K/V run ahead
 * of the dependency chain through a TMA ring, and hands activations from step to step through the clusters'
 * shared memory and counters in L2 instead of one kernel per projection.  It computes the same quantities with
 * the same rounding points.  Its clusters have 8 CTAs where the device can hold one per head at once, else 6.
 * enable = 0 (the default): kernel-per-step path, which is the faster one on the devices measured so far;
 * 1: the persistent kernel with the cluster size the library chooses; 6 or 8: that cluster size where it fits.
 * Host-side switch: takes effect with the next call. */
vadusa_status vadusa_set_fused_pass(vadusa_ctx *ctx, int32_t enable);
/* How many of that kernel's clusters (one per head, of the chosen size) the device can hold at once, as found
 * when the first such pass was enqueued (-1 before).  The persistent kernel is used only if this is >= n_heads. */
int32_t vadusa_fused_pass_clusters(const vadusa_ctx *ctx);

/* ---- sampler hook (paper Sec. II-C, last paragraph) ----------------------------------------
 * The paper notes that improved sampling strategies (e.g. avoiding repetitions) are used by taking
 * their outcomes as the predictions of the original head, with the tau draws made by the same
 * strategy.  The strategies this hook serves are those that reshape the base head's distribution
 * per sequence: bias is fp32 [batch][ld] (ld >= vocab) in device memory, owned by the caller, and
 * is added (one fp32 addition, before temperature, nucleus and noise) to every base-head logits
 * row of the sequence wherever it is sampled: the root, the tau draws of Algorithm 1 and the next
 * root.  -inf bans a token.  The draft heads and the returned logits are not changed.  The caller
 * may rewrite the table between iterations (stream-ordered); NULL switches the hook off.  The
 * pointer is read by the kernels of later calls; it must stay valid until replaced. */
vadusa_status vadusa_set_logit_bias(vadusa_ctx *ctx, const float *bias, int32_t ld);

/* ---- sparse-tree construction (paper Sec. II-D) --------------------------------------
 * The paper grows its sparse candidate tree greedily so as to maximise the expected accepted
 * length within a fixed number of nodes, from acceptance probabilities measured with the
 * full tree.
 *
 * vadusa_accept_stats: since the last reset, how often the acceptance test (Algorithm 1) was
 * applied to a candidate of draft head j+1 with top-k rank r below an accepted parent
 * (h_tested[j * VADUSA_MAX_DRAFT_TOPK + r]) and how often it passed (h_accepted[...]); host
 * int64 arrays of VADUSA_MAX_DEPTH * VADUSA_MAX_DRAFT_TOPK entries.  Iterations with a forced
 * winner are not counted.  Synchronises; reset != 0 clears the counters afterwards.
 *
 * vadusa_build_sparse_tree (host only, no GPU): h_prob[j * topk + r] = probability that the
 * rank-r candidate of head j+1 is accepted given that its parent is (j < depth, r < topk).  A
 * node's probability is the product along its root path; starting from the root, the candidate
 * child with the highest probability is added n_nodes - 1 times (ties: shallower, then
 * lexicographically smaller rank path).  Writes parent[] and rank[] in (depth, rank path)
 * order, ready for vadusa_set_tree, and the expected accepted length 1 + sum of the node
 * probabilities.  VADUSA_EINVAL if the capped tree has fewer than n_nodes nodes. */
vadusa_status vadusa_accept_stats(vadusa_ctx *ctx, int64_t *h_tested, int64_t *h_accepted, int32_t reset);
vadusa_status vadusa_build_sparse_tree(const double *h_prob, int32_t depth, int32_t topk, int32_t n_nodes,
                                       int32_t *h_parent, int32_t *h_rank, double *h_expected_len);

/* ---- fitting the draft heads (paper Sec. II-A, III-A.2) -----------------------------------
 * "The i-th draft head is responsible for predicting the (i+1)-th next token by the supervision of a
 * cross-entropy loss multiplied with lambda^i" (i >= 1), with the base model fixed (the paper's "wot" setting:
 * lambda 0.8, learning rate 0.002, 40 warm-up steps).  The paper names no optimiser and no normalisation:
 * here every head's cross-entropy is averaged over the positions that have a target, the optimiser is Adam
 * (beta 0.9 / 0.999, eps 1e-8, no weight decay), and the learning rate rises linearly over the warm-up steps.
 * Not part of the decoding path: plain fp32 arithmetic on fp32 master copies of the heads kept in `state`
 * (device memory owned by the caller, >= vadusa_fit_state_bytes(cfg, max_tokens), 256-byte aligned).
 * vadusa_fit_begin copies the heads from the weight blob; every vadusa_fit_step writes the updated heads
 * back INTO THE CALLER'S WEIGHT BLOB (tensors "draft<i>.w/.b/.u", in the model dtype), so the next
 * vadusa_draft uses them.
 *   hidden  [n_tokens][d_model] in the model dtype: final-LayerNorm outputs of the frozen base model at
 *           consecutive positions (vadusa_set_prefill_tap makes vadusa_prefill deliver them)
 *   targets int32 [n_tokens][n_draft_heads]: targets[t][i] = the token at position t + 2 + i (the (i+2)-th
 *           token after position t's own; head numbering from 0), or -1 where the stream has none
 *   loss_out device fp32 [1 + n_draft_heads] or NULL: the weighted total, then each head's mean cross-entropy
 * Work is enqueued on the context's stream; no call synchronises. */
int64_t vadusa_fit_state_bytes(const vadusa_config *cfg, int32_t max_tokens);
vadusa_status vadusa_fit_begin(vadusa_ctx *ctx, void *state, int64_t state_bytes, int32_t max_tokens, float lambda,
                               float learning_rate, int32_t warmup_steps);
vadusa_status vadusa_fit_step(vadusa_ctx *ctx, const void *hidden, const int32_t *targets, int32_t n_tokens,
                              float *loss_out);
vadusa_status vadusa_fit_end(vadusa_ctx *ctx);
/* While set, vadusa_prefill also stores the final-LayerNorm output of every prefix token it scores:
 * hidden_out [batch][stride][d_model] in the model dtype, row (b, s) for token s of the prefix passed in that
 * call (stride >= the longest prefix).  NULL switches it off. */
vadusa_status vadusa_set_prefill_tap(vadusa_ctx *ctx, void *hidden_out, int32_t stride);

/* ---- measurement ------------------------------------------------------------------ */
/* Between vadusa_profile_begin and vadusa_profile_end every kernel launch of the library
 * is bracketed by a pair of CUDA events on the context's stream.  vadusa_profile_end
 * synchronises and returns, per kernel class, the number of launches and the summed
 * device time.  h_out: host array of `capacity` >= 16 entries; *h_count entries are
 * written.  The events perturb the stream slightly: take whole-step timings outside. */
typedef struct {
  char name[32];
  int64_t launches;
  double total_ms;
} vadusa_kernel_time;
vadusa_status vadusa_profile_begin(vadusa_ctx *ctx);
vadusa_status vadusa_profile_end(vadusa_ctx *ctx, vadusa_kernel_time *h_out, int32_t capacity, int32_t *h_count);

/* ---- for callers that cannot allocate device memory ---------------------------------- */
/* (The paper has no counterpart to this call; it exists for deployment reasons only.)
 * The draft heads' top-k, like the draft-head part of vadusa_draft, but without a context
 * and without a workspace: the intermediate results (the residual-block outputs and the
 * heads' logits) live in a fixed 2 MiB device array compiled into the library, which every
 * GPU that loads the library holds until the process exits.  It is meant for code that may
 * not call cudaMalloc: a plug-in inside another framework's memory plan, a real-time audio
 * loop that must not touch the allocator once it runs, a process whose device memory was
 * handed out completely before this library was loaded.  The call itself allocates nothing,
 * on the host or on the device; but the FIRST call on a device makes the CUDA runtime load this
 * part of the library and reserve the 2 MiB array there, which fails (VADUSA_ECUDA) if the
 * device has no memory left: make one call at start-up, before memory is handed out.
 *   draft_w [heads][d_model][d_model], draft_u [heads][ceil(vocab/128)*128][d_model] in the
 *   model dtype (0 fp32, 1 bf16; the layout of the weight blob), draft_b fp32 [heads][d_model],
 *   hstar [batch][d_model] in the model dtype, topk_out int32 [batch][heads][topk]; all device
 *   memory of the current device.  Work is enqueued on `stream`; the call does not synchronise.
 * Limits: batch <= 64 and heads * batch * (d_model * sizeof(dtype) + ceil(vocab/128)*128 * 4)
 *   + 768 <= vadusa_static_scratch_bytes(); larger requests return VADUSA_ENOMEM with a message
 *   in vadusa_static_last_error().  The arithmetic is the plain-FMA one for both dtypes.
 * The first call on a device looks up the array's device address (with that device current):
 *   make that first call outside any stream capture.
 * All calls on one GPU share the array and it keeps what the last call left there; every
 *   call overwrites what it reads, so nothing needs clearing, but two calls that overlap on
 *   the GPU (different streams, no ordering between them) race on it.
 * On the host the call and vadusa_static_last_error() share unsynchronised state (the per-device
 *   address table and the message buffer): call them from one thread at a time. */
vadusa_status vadusa_draft_topk_static(const void *draft_w, const float *draft_b, const void *draft_u,
                                       const void *hstar, int32_t dtype, int32_t batch, int32_t d_model,
                                       int32_t vocab, int32_t n_draft_heads, int32_t topk, int32_t eos_masked,
                                       int32_t *topk_out, void *stream);
int64_t vadusa_static_scratch_bytes(void);
const char *vadusa_static_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* VADUSA_H */
