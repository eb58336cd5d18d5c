/*
 * dream.h — C ABI of the DREAM draft-and-verify hot path for NVIDIA B200 (sm_100a).
 *
 * One library, one GPU, one CUDA stream per context.  The calls follow the paper's
 * statement of the problem (DREAM, arXiv 2505.19201): a target VLM decoder M_ta with L
 * blocks processes q text tokens and v visual tokens (Section 3); a one-layer draft
 * model M_da cross-attends to cached target features over a compressed set of visual
 * tokens (Section 3.1, Eq. 1; Section 3.3) and expands a token tree (Section 3.1, tree
 * drafting); the target verifies the tree in one masked pass and the longest matching
 * path is accepted (Section 2.1; Section 4, evaluation setup).
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory addresses valid on the context's device;
 *     "host" pointers are ordinary process memory.  Every pointer says which it is.
 *   - Every matrix is row-major [out_features, in_features] ("weight-stationary" layout:
 *     one output feature is one contiguous row), element type = config.dtype.
 *   - The library allocates nothing on the device: the caller passes one arena of
 *     dream_arena_bytes() bytes to dream_init and owns it; weights and in/out buffers are
 *     the caller's too and are only borrowed (weights for the context's lifetime).
 *   - Calls enqueue work on the context's stream and return; outputs are device buffers
 *     and are ready when the stream reaches that point.  Only dream_step_host and
 *     dream_poll synchronise.
 *   - Errors: argument and state checks happen on the host before anything is enqueued
 *     and leave the context untouched; the code is returned and a message is kept for
 *     dream_last_error.  Device-side anomalies (a bounded wait that expired, an index out
 *     of range) never trap: they set a status word that dream_poll reports.
 *   - Not thread-safe: one thread drives one context.
 *   - Call order: dream_init -> per sequence { dream_prefill -> dream_compress_visual }
 *     -> loop { dream_draft_tree -> dream_verify_tree -> dream_accept }.
 */
#ifndef DREAM_H_
#define DREAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dream_ctx dream_ctx;
typedef int32_t dream_status;

enum {
  DREAM_OK = 0,
  DREAM_E_ARG = -1,            /* bad argument (null, out of range, misaligned) */
  DREAM_E_STATE = -2,          /* call out of order for this sequence */
  DREAM_E_NOMEM = -3,          /* arena too small */
  DREAM_E_CAPACITY = -4,       /* sequence would outgrow max_seq / max_prompt / page pool */
  DREAM_E_CUDA = -5,           /* a CUDA runtime or driver call failed */
  DREAM_E_DEVICE_TIMEOUT = -6, /* a bounded device-side wait expired */
  DREAM_E_UNSUPPORTED = -7     /* shape or dtype outside what the kernels handle */
};
enum { DREAM_F32 = 0, DREAM_BF16 = 1 };
enum { DREAM_TAP_FIXED = 0, DREAM_TAP_ENTROPY_MIN = 1, DREAM_TAP_ENTROPY_MAX = 2 };

/* Shapes and hyper-parameters; plain data, copied by dream_init. */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab;   /* d_model <= 16384 */
  int32_t dtype;                 /* DREAM_F32 or DREAM_BF16: weights, KV caches, GEMM inputs */
  float rms_eps, rope_theta;
  int32_t max_batch;             /* sequences resident at once */
  int32_t max_seq;               /* verified tokens per sequence, upper bound */
  int32_t max_prompt;            /* q + v upper bound for dream_prefill */
  int32_t max_visual;            /* v upper bound */
  int32_t page_tokens;           /* tokens per target-KV page (power of two, 16..256) */
  int32_t tree_depth, tree_topk, tree_beam, tree_max_nodes;   /* D, K, beam width, N */
  int32_t tap_mode, tap_layer, tap_lo, tap_hi;   /* 1-based layers; [lo,hi] = entropy search range */
  int32_t score_include_self;    /* 1: a token's attention to itself counts in its importance */
  int32_t xattn_full_memory;     /* 1: cross-attention memory keeps all n prompt positions */
  int32_t draft_blocks;          /* 0 or 1: one draft layer (self-attention, Eq. 1, MLP); 3: the three
                                    blocks of Section 4 (initial decoder block, Eq. 1 block, final decoder block) */
  int32_t track_entropy;         /* 1: keep Eq. 2 up to date while decoding (dream_layer_entropy); 0: prefill only */
} dream_config;

/* Target weights (device, borrowed).  Arrays of n_layers device pointers live on the HOST. */
typedef struct {
  const void *embed;             /* [vocab, d_model] */
  const void *const *ln1;        /* each [d_model] */
  const void *const *wqkv;       /* each [(n_heads + 2 n_kv_heads) head_dim, d_model]: Q rows, K rows, V rows */
  const void *const *wo;         /* each [d_model, n_heads head_dim] */
  const void *const *ln2;        /* each [d_model] */
  const void *const *wgu;        /* each [2 d_ff, d_model]: gate rows then up rows */
  const void *const *wd;         /* each [d_model, d_ff] */
  const void *ln_f;              /* [d_model] */
  const void *lm_head;           /* [vocab, d_model] */
} dream_target_weights;

/* Draft weights (device, borrowed): one layer = self-attention, cross-attention, MLP.
 * The draft shares the target's embedding, final norm and LM head.
 * With draft_blocks = 3 (Section 4: an initial decoder block, an intermediate cross-attention
 * block, a final decoder block, each pre-norm with a gated MLP) the first group is the initial
 * block's attention and i_* its MLP; lnx..xo and ln2, wgu, wd are the intermediate block; f_* is the
 * final block.  The i_* and f_* pointers are ignored (may be NULL) otherwise. */
typedef struct {
  const void *ln1, *wqkv, *wo;           /* self-attention, shapes as in the target */
  const void *lnx, *xq, *xkv, *xo;       /* cross-attention (Eq. 1): xq [H hd, d], xkv [2 H_kv hd, d] (K rows then V rows), xo [d, H hd] */
  const void *ln2, *wgu, *wd;            /* fusion MLP */
  const void *i_ln2, *i_wgu, *i_wd;      /* draft_blocks = 3: MLP of the initial block */
  const void *f_ln1, *f_wqkv, *f_wo;     /* draft_blocks = 3: self-attention of the final block */
  const void *f_ln2, *f_wgu, *f_wd;      /* draft_blocks = 3: MLP of the final block */
} dream_draft_weights;

/* A token tree, caller-allocated DEVICE buffers of capacity tree_nodes = dream_tree_nodes().
 * Node 0 is the root (the pending token); parents precede children. */
typedef struct {
  int32_t *tokens;               /* [T] */
  int32_t *parent;               /* [T], parent[0] = -1 */
  int32_t *depth;                /* [T], depth[0] = 0 */
  uint32_t *mask;                /* [T][4] ancestor-or-self bit set, bit j of word j/32 */
  float *cum_logp;               /* [T] cumulative draft log-probability; may be NULL on input */
} dream_tree;

/* Number of tree nodes T = 1 + min(N, candidates) for this configuration (Section 4:
 * depth, children per node, maximum draft length).  Host-only arithmetic. */
dream_status dream_tree_nodes(const dream_config *cfg, int32_t *T);

/* Depths and ancestor-or-self bit masks of a tree given by its parent array (Section 3.1: the
 * tree mask lets a node attend to its ancestors only): node 0 is the root, parent[0] = -1 and
 * every other node's parent has a smaller index.  All four arrays are HOST memory: parent
 * int32[n_nodes] in; depth int32[n_nodes] and mask uint32[n_nodes][4] out, in the layout of
 * dream_tree.  For callers that inject their own trees into dream_verify_tree.  Host-only
 * arithmetic; DREAM_E_ARG for a parent that does not precede its child or n_nodes outside 1..128. */
dream_status dream_tree_from_parents(const int32_t *parent, int32_t n_nodes, int32_t *depth, uint32_t *mask);

/* Bytes of device memory dream_init needs for this configuration.  Host-only. */
dream_status dream_arena_bytes(const dream_config *cfg, size_t *bytes);

/* Create a context.  arena: device, >= dream_arena_bytes, 256-byte aligned, zeroed by the
 * library.  cuda_stream: a cudaStream_t (NULL = legacy default stream).  Weights are
 * borrowed until dream_free.  The problem set-up of Section 3: one M_ta, one M_da. */
dream_status dream_init(const dream_config *cfg, const dream_target_weights *tw,
                        const dream_draft_weights *dw, void *arena, size_t arena_bytes,
                        void *cuda_stream, dream_ctx **out);

/* Target prefill over the n = q + v prompt (Section 3: M_ta processes all q + v inputs and
 * emits t_{n+1}).  The sequence holds visual_embeds (device, [v, d_model], dtype) at
 * positions [vis_start, vis_start + v) and embed[prompt_ids] (device int32 [q]) elsewhere.
 * Also computes the average attention entropy of every layer (Eq. 2) and selects the
 * feature-tap layer l* per config.tap_mode (Section 3.2).  Outputs (device, may be NULL):
 * first_token int32[1], first_margin float[1] (top-1 minus top-2 logit),
 * layer_entropy float[n_layers], tap_layer int32[1] (1-based). */
dream_status dream_prefill(dream_ctx *ctx, int32_t seq, const void *visual_embeds, int32_t v,
                           int32_t vis_start, const int32_t *prompt_ids, int32_t q,
                           int32_t *first_token, float *first_margin, float *layer_entropy,
                           int32_t *tap_layer);

/* Override l* of a prefilled sequence (1-based) before dream_compress_visual. */
dream_status dream_set_tap(dream_ctx *ctx, int32_t seq, int32_t tap_layer);

/* Visual-token compression (Section 3.3): importance of visual token j = attention it
 * receives at layer l* summed over query rows and heads; the k highest are kept.  Builds
 * the draft's compressed context (self-attention K/V from input embeddings, cross-attention
 * memory from the tapped features S^{l*}, Eq. 1).  With draft_blocks = 3 the draft then runs
 * over the compressed context (the reduced sequence of Section 3.3): a row at position p attends
 * causally in both decoder blocks and, in the Eq. 1 block, to the memory rows of positions < p;
 * what stays are the K/V rows of the initial and of the final block.  forced_idx (device
 * int32[k], ascending, or NULL) replaces the selection.  Outputs (device, may be NULL): kept_idx
 * int32[k] ascending, scores float[v]. */
dream_status dream_compress_visual(dream_ctx *ctx, int32_t seq, int32_t k,
                                   const int32_t *forced_idx, int32_t *kept_idx, float *scores);

/* Draft a token tree for each listed sequence (Section 3.1): D passes of the draft layer
 * (self-attention over the draft cache, cross-attention over target features plus the
 * draft's own earlier features, fusion MLP), top-K expansion per pass, beam selection, and
 * a final re-rank to T nodes.  With draft_blocks = 3 a pass is the three blocks of Section 4, and
 * the tokens the last acceptance emitted run through them first (with the memory rows of earlier
 * positions) to leave their K/V rows in both decoder blocks' caches.  seqs: HOST int32[n_seqs], distinct.  trees: HOST array of
 * n_seqs dream_tree structs whose members are DEVICE buffers that receive the trees. */
dream_status dream_draft_tree(dream_ctx *ctx, const int32_t *seqs, int32_t n_seqs,
                              const dream_tree *trees);

/* Tree-masked verification by the target (Section 3.1: the same tree mask is used during
 * verification): the T tree tokens of each sequence run through all L blocks, node i at
 * position P + depth[i], attending to the verified prefix and to its ancestors' rows.
 * Outputs (device): node_argmax int32[n_seqs][T]; node_margin float[n_seqs][T] or NULL;
 * logits float[n_seqs][T][vocab] or NULL. */
dream_status dream_verify_tree(dream_ctx *ctx, const int32_t *seqs, int32_t n_seqs,
                               const dream_tree *trees, int32_t *node_argmax,
                               float *node_margin, float *logits);

/* Greedy acceptance and state update (Section 2.1; Section 4: one extra target token per
 * round): follows from the root the child whose token equals its parent's argmax; emits
 * the A accepted tokens plus the target's own next token; compacts the target KV cache so
 * the accepted path occupies positions P..P+A; appends the accepted rows' tapped features
 * to the cross-attention memory; P += A + 1.  seqs and trees must be those of the last
 * dream_verify_tree, in the same order (DREAM_E_STATE otherwise: the verify's tapped features and
 * row map are kept by position in that list).  Outputs (device): accept_len int32[n_seqs];
 * out_tokens int32[n_seqs][D+1] (first A+1 valid); compaction_src int32[n_seqs][D+1] (tree
 * node whose KV row moved to P+j; first A+1 valid). */
dream_status dream_accept(dream_ctx *ctx, const int32_t *seqs, int32_t n_seqs,
                          const dream_tree *trees, const int32_t *node_argmax,
                          int32_t *accept_len, int32_t *out_tokens, int32_t *compaction_src);

/* Acceptance at a sampling temperature above zero, and the same state update as dream_accept
 * (Section 2.1: a draft token d is accepted with probability min(1, P_target(d) / P_draft(d)), a
 * rule that holds at any temperature; Section 4 reports Temp = 1).  The tree's children are the
 * draft's top-K choices, so each is a point-mass proposal (P_draft = 1): child c of the current
 * node, tried in node order, is kept when u < p(token_c), where p = softmax(logits[cur] /
 * temperature) without the tokens already refused at this node, renormalised.  When every child
 * is refused, or the node has none, the emitted token is drawn from what is left of p by
 * inverting its cumulative sum in token order.  The emitted tokens follow the target's own
 * sampling distribution whatever the tree proposed.
 *   logits      : device float [n_seqs][T][vocab], e.g. the dump of dream_verify_tree
 *   temperature : > 0 (DREAM_E_ARG otherwise)
 *   uniforms    : device float [n_seqs][D+1][T], numbers in [0, 1) drawn by the caller: [b][j][r]
 *                 decides the r-th child tried at path step j, [b][j][T-1] is the final draw
 * Outputs as in dream_accept.  Follows dream_verify_tree (DREAM_E_STATE otherwise); enqueues on the
 * context's stream and returns. */
dream_status dream_accept_sample(dream_ctx *ctx, const int32_t *seqs, int32_t n_seqs,
                                 const dream_tree *trees, const float *logits, float temperature,
                                 const float *uniforms, int32_t *accept_len, int32_t *out_tokens,
                                 int32_t *compaction_src);

/* One whole round (draft, verify, accept) with HOST result buffers: runs the three calls
 * above on the context's internal tree buffers, copies accept_len [n_seqs] and out_tokens
 * [n_seqs][D+1] to host memory and waits for them.  This is the call a serving loop makes. */
dream_status dream_step_host(dream_ctx *ctx, const int32_t *seqs, int32_t n_seqs,
                             int32_t *accept_len_host, int32_t *out_tokens_host);

/* Read back per-sequence state (host outputs; synchronises the stream).  The host bounds a
 * sequence's verified length from above between read-backs (it grows by at most tree_depth + 1 per
 * round); this call, dream_step_host, and a small asynchronous copy behind every acceptance make
 * the bound exact again, so DREAM_E_CAPACITY is only reported when max_seq is really reached. */
dream_status dream_seq_state(dream_ctx *ctx, int32_t seq, int32_t *verified_len,
                             int32_t *pending_token, int32_t *tap_layer);

/* Eq. 2 over the rows verified so far (Section 3.2 speaks of selecting the layer "during each
 * decoding step"): with config.track_entropy = 1 the verification also leaves every tree row's
 * attention entropy per layer and head, and dream_accept adds those of the accepted path to the
 * per-layer sums of the prefill, so nothing is recomputed.  Outputs (HOST, may be NULL):
 * layer_entropy float[n_layers] = AE(l) over the verified_len rows; layer_now = the layer
 * config.tap_mode would select from it now (1-based; the fixed layer for DREAM_TAP_FIXED).  The
 * draft keeps the layer chosen at prefill (its memory holds that layer's features); this call only
 * reports.  Synchronises the stream.  DREAM_E_STATE when track_entropy is 0 or the sequence has no
 * prefill. */
dream_status dream_layer_entropy(dream_ctx *ctx, int32_t seq, float *layer_entropy, int32_t *layer_now);

/* Debug read-back of internal device buffers for parity tests (synchronises).  what:
 * 0 = target K row [n_kv_heads*head_dim] of (layer, position) as float,
 * 1 = target V row, 2 = cross-memory K row (index = memory row), 3 = cross-memory V row,
 * 4 = draft self-attention K row, 5 = draft self-attention V row,
 * 6 = tapped features of tree node `index` from the last verify [d_model],
 * 7 = final hidden state of tree node `index` from the last verify [d_model],
 * 8 = K row of the draft's final decoder block (draft_blocks = 3), 9 = its V row.
 * dst: HOST float buffer. */
dream_status dream_debug_read(dream_ctx *ctx, int32_t seq, int32_t what, int32_t layer,
                              int32_t index, float *dst);

/* Test hook: out[r][c] = sum_k X[r][k] W[c][k] through the context's GEMM path (the same
 * kernels every projection of the model uses).  W: device [N][K] in config.dtype; X: device
 * float [rows][K]; out: device float [rows][N]; rows <= 256 (128 for bf16 with split == 0);
 * K <= max(d_model, d_ff); bf16: K a multiple of 64, N of 8.  split != 0 feeds bf16 inputs as a
 * high and a low bf16 row per token. */
dream_status dream_debug_gemm(dream_ctx *ctx, const void *W, const float *X, int32_t rows,
                              int32_t N, int32_t K, int32_t split, float *out);

/* How many GEMM launches so far went to the tensor-core kernel and to the CUDA-core kernel. */
dream_status dream_gemm_counts(const dream_ctx *ctx, int64_t *tensor_core, int64_t *cuda_core);

/* Per-launch timing of the weight-streaming GEMM, the kernel that moves nearly all of a step's
 * bytes (Section 4 reports whole-step speed only; this is the measurement hook for the kernel's
 * bandwidth).  on != 0: from now on every tensor-core GEMM launch is bracketed by two CUDA events
 * on the context's stream (up to 8192 launches; the brackets keep neighbouring kernels from
 * overlapping it, so use it in a pass of its own).  on == 0: stop, wait for the stream and
 * return the number of timed launches, the sum of their durations in milliseconds and the
 * weight bytes they streamed (HOST outputs, may be NULL). */
dream_status dream_gemm_timing(dream_ctx *ctx, int32_t on, int64_t *launches, double *total_ms,
                               double *weight_bytes);

/* Top-k and log-sum-exp of a logits matrix with no arena and no allocation.  The paper has no
 * counterpart to this call; it exists for callers that are not allowed to allocate device memory:
 * a serving process that froze its memory pool after start-up, a plug-in that only gets the
 * buffers its host hands it, or code that must not call cudaMalloc because that call
 * synchronises the whole device.  It runs the library's k_topk_lse kernel (the one behind the
 * LM heads of dream_draft_tree and dream_verify_tree) on a caller-owned matrix.
 *   logits : device float [rows][vocab], row-major, 16-byte aligned
 *   outputs: device top_val float [rows][ktop] (descending; equal values -> lower id first),
 *            top_id int32 [rows][ktop], lse float [rows]
 *   cuda_stream: a cudaStream_t of the current device (NULL = legacy default stream)
 * The kernel's scratch (partial lists and counters) is a fixed ~1.1 MB array built into the
 * library, held by every GPU that loads it until the process ends.  Limits: rows <= 128,
 * vocab <= 262144, ktop <= 16; larger sizes return DREAM_E_CAPACITY and enqueue nothing.  The
 * first call on each device looks the array's device address up (no allocation); make that call
 * with the device current and before any stream capture.  All calls share the one array: it
 * keeps the previous call's contents (the call clears the counters it needs at zero), and two
 * calls whose kernels can overlap on the GPU (different streams, no ordering between them) race
 * on it and give wrong results, so order them.  Asynchronous like the other calls; errors are
 * reported through dream_last_error(NULL). */
dream_status dream_topk_lse_static(const float *logits, int32_t rows, int32_t vocab, int32_t ktop,
                                   float *top_val, int32_t *top_id, float *lse, void *cuda_stream);

/* Timeline of the context's stream (a measurement hook; Section 4 times whole steps only).
 * buffer: DEVICE array of 2 + 2 * capacity_entries 64-bit words, or NULL to stop tracing.  While
 * installed, every kernel of the library appends (kernel id, nanosecond timer) at the moment its
 * predecessor in the stream has completed; word 0 counts the entries.  Differences between
 * consecutive entries give each kernel's time on the critical path, overlap included.  The
 * buffer is process-wide (one traced context at a time).  Synchronises the stream. */
dream_status dream_trace(dream_ctx *ctx, unsigned long long *buffer, int64_t capacity_entries);

/* Name of a kernel id found in a trace buffer.  Host-only. */
const char *dream_trace_name(int32_t id);

/* Forget a sequence (its pages return to the pool). */
dream_status dream_seq_reset(dream_ctx *ctx, int32_t seq);

/* Wait for the stream and report the device status word: DREAM_OK, DREAM_E_DEVICE_TIMEOUT (a
 * bounded wait inside a kernel ran out) or DREAM_E_STATE (a kernel met a malformed tree, an index
 * or a capacity out of range, or a logits row without mass; the offending rows were skipped).
 * The word is sticky: it is not cleared by reading it. */
dream_status dream_poll(dream_ctx *ctx);

/* Number of kernels this context has launched since dream_init. */
int64_t dream_launch_count(const dream_ctx *ctx);

/* Message of the last failed call on this context (or of the last failed dream_init when
 * ctx is NULL).  The string is owned by the library. */
const char *dream_last_error(const dream_ctx *ctx);

/* Destroy the context.  The arena and the weights stay the caller's. */
void dream_free(dream_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* DREAM_H_ */
