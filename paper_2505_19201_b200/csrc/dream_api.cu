// C ABI of the DREAM draft-and-verify hot path: context, arena layout, and the host-side
// sequences of kernel launches behind each entry point.  Everything the entry points
// compute runs in the kernels of this library; the host only validates and enqueues.
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "../../include/dream.h"
#include "attn.cuh"
#include "attn_merge.cuh"
#include "attn_tc.cuh"
#include "colsum_tc.cuh"
#include "common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "rows.cuh"
#include "tree.cuh"

#define AM_MAX_CHUNKS 32        // most key chunks the split-K attention cuts a sequence into
#define ROW_CHUNK 256          // most rows any launch set holds (max_batch * tree nodes, a prefill chunk)

#define SNAP_SLOTS 4

enum { PH_EMPTY = 0, PH_PREFILLED, PH_READY, PH_DRAFTED, PH_VERIFIED };

static char g_init_error[256];

struct dream_ctx {
  dream_config cfg;
  cudaStream_t stream;
  TreeShape ts;
  int T, esz, qkvN, Hhd, kvN, n_cand, tap_lo_eff, cap_rows, pps, n_pages, RM, XR, gemm_rows_lm;
  int use_tc, use_pdl, gemm_failed;
  cudaError_t launch_err;              // first refused kernel launch of the call being enqueued
  const char *launch_err_name;
  int chunk;                           // prompt rows per pass of the prefill loop
  double *rope_inv;                    // [head_dim / 2] rotary inverse frequencies
  float2 *rope_tab;                    // [ROW_CHUNK][head_dim / 2] rotary (cos, sin) of the rows of the call being enqueued
  std::vector<const void *> ln1, wqkv, wo, ln2, wgu, wd;
  const void *embed, *ln_f, *lm_head;
  dream_draft_weights dw;
  // arena
  char *arena;
  size_t arena_bytes;
  void *kv_pool;
  long long kv_stride, layer_stride;
  int *page_table, *status;
  SeqDev sd;
  float *dself, *dmem;
  float *dself2;                       // three-block draft: K/V rows of the final decoder block (else null)
  bool three;                          // cfg.draft_blocks == 3
  DraftTreeDev dt;
  TreePtrs itree[DREAM_MAX_BATCH];
  RowMeta rm[2];
  int *gather_idx, *ctx_pos, *flags;
  uint32_t *vmask;
  void *qbuf;                          // query rows, 4 bytes per element (see q_store4)
  float *x, *x0, *gout, *lse_pre, *ent_pre, *ae, *scores_all, *taps_store, *tapbuf;
  void *xn, *raw, *act, *attn_out;
  float *top_val, *lse_rows, *margin_i;
  TopkScratch tks;
  float *am_part_o, *am_part_ml;       // split-K attention partials
  // track_entropy: the chunks' u beside am_part_ml, every tree row's entropy [layer][ROW_CHUNK][H] from
  // the last verification, and the per-layer sums over the verified rows [seq][layer]
  float *am_part_u, *row_ent, *ent_sum;
  int am_rt_max;
  int key_ub0[DREAM_MAX_BATCH];        // permanent rows of the draft caches right after compression
  // Verified lengths as the host knows them.  The device advances P by A + 1 per accept and the host
  // only knows A <= D, so p_ub grows by D + 1 per accept until a snapshot of the device's P arrives:
  // every accept enqueues a small copy of P into pinned memory behind an event, and the next call
  // that plans launches adopts the newest snapshot whose event has completed (no host wait).
  int *h_snap;                         // pinned [SNAP_SLOTS][DREAM_MAX_BATCH]
  cudaEvent_t snap_ev[SNAP_SLOTS];
  int snap_busy[SNAP_SLOTS];           // an event was recorded for this slot and not yet seen complete
  long long snap_accepts[SNAP_SLOTS][DREAM_MAX_BATCH], snap_epoch[SNAP_SLOTS][DREAM_MAX_BATCH];
  long long snap_order[SNAP_SLOTS], snap_clock;
  long long accepts[DREAM_MAX_BATCH], epoch[DREAM_MAX_BATCH];
  int last_verify_n, last_verify_seq[DREAM_MAX_BATCH];   // the sequence list of the last dream_verify_tree
  int cur_seq[DREAM_MAX_BATCH];        // sequences of the call being enqueued, by slot
  int tk_nsplit, tk_nv;                // vocabulary blocks of the top-k kernel, columns per thread (4 or 16)
  int *top_id, *argmax_i, *accept_len_i, *out_tokens_i, *comp_src_i;
  size_t gout_floats;
  // host side
  int phase[DREAM_MAX_BATCH], n_prompt[DREAM_MAX_BATCH], p_ub[DREAM_MAX_BATCH];
  int prefill_seq;                     // sequence whose prefill scratch is live (-1 none)
  int pf_v, pf_vis_start, pf_q;
  std::vector<int> free_pages;
  std::vector<int> seq_pages[DREAM_MAX_BATCH];
  int *h_stage;                        // pinned: page-table staging + step_host results
  long long launches, tc_launches, simt_launches;
  GemmTcPlan tc;
  AtMapCache at_maps;
  // per-launch timing of the weight-streaming GEMM (dream_gemm_timing)
  int prof_on, prof_n;
  double prof_bytes;
  std::vector<cudaEvent_t> prof_ev;
  char err[256];
};

static dream_status fail(dream_ctx *c, dream_status code, const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(c ? c->err : g_init_error, 256, fmt, ap);
  va_end(ap);
  return code;
}

#define CUDA_OK(c, call)                                                              \
  do {                                                                                \
    cudaError_t e_ = (call);                                                          \
    if (e_ != cudaSuccess) return fail(c, DREAM_E_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

// End of an entry point that enqueued kernels: report a refused launch by name.
static dream_status call_done(dream_ctx *c) {
  if (c->launch_err != cudaSuccess) {
    cudaError_t e = c->launch_err;
    c->launch_err = cudaSuccess;
    cudaGetLastError();
    return fail(c, DREAM_E_CUDA, "launch of %s failed: %s", c->launch_err_name, cudaGetErrorString(e));
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(c, DREAM_E_CUDA, "CUDA error after enqueueing: %s", cudaGetErrorString(e));
  if (c->gemm_failed) { c->gemm_failed = 0; return fail(c, DREAM_E_CUDA, "a GEMM launch was refused (shape, output room or tensor map)"); }
  return DREAM_OK;
}

// Every kernel is launched with programmatic stream serialization: it may become resident while
// its predecessor still runs and blocks in pdl_wait() until that one has finished.
// A refused launch is remembered with the kernel's name (the first one of a call); the entry point
// that enqueued it reports it through call_done().
template <typename... P, typename... A>
static inline void launch_k(dream_ctx *c, const char *name, void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = c->use_pdl ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
  if (e != cudaSuccess && c->launch_err == cudaSuccess) { c->launch_err = e; c->launch_err_name = name; }
  c->launches++;
}
#define LAUNCH(c, kernel, grid, block, smem, ...) launch_k(c, #kernel, kernel, dim3(grid), dim3(block), (size_t)(smem), __VA_ARGS__)
#define TOPK_LAUNCH(c, grid, ...)                                                        \
  do {                                                                                   \
    if ((c)->tk_nv == 4) LAUNCH(c, (k_topk_lse<4>), grid, TOPK_THREADS, 0, __VA_ARGS__); \
    else LAUNCH(c, (k_topk_lse<16>), grid, TOPK_THREADS, 0, __VA_ARGS__);                \
  } while (0)

// ------------------------------------------------------------------------------------- shapes

static int tree_shape(const dream_config *cfg, TreeShape *ts) {
  int D = cfg->tree_depth, K = cfg->tree_topk, bw = cfg->tree_beam, N = cfg->tree_max_nodes;
  if (D < 1 || D > DREAM_MAX_DEPTH || K < 1 || K > TOPK_MAX || bw < 1 || N < 1) return -1;
  memset(ts, 0, sizeof(*ts));
  ts->D = D; ts->K = K; ts->N = N;
  ts->beam[0] = 1; ts->in_off[0] = 0; ts->cand_off[0] = 0;
  int ni = 1, nc = 0;
  for (int p = 1; p <= D; ++p) {
    int created = ts->beam[p - 1] * K;
    if (created > 256) return -1;
    nc += created;
    ts->cand_off[p] = nc;
    ts->beam[p] = created < bw ? created : bw;
    ts->in_off[p] = ni;
    if (p < D) ni += ts->beam[p];
  }
  ts->NI = ni; ts->NC = nc;
  ts->T = 1 + (N < nc ? N : nc);
  if (ni > 64 || ts->T > 128) return -1;
  return 0;
}

extern "C" dream_status dream_tree_nodes(const dream_config *cfg, int32_t *T) {
  TreeShape ts;
  if (!cfg || !T) return fail(nullptr, DREAM_E_ARG, "null argument");
  if (tree_shape(cfg, &ts)) return fail(nullptr, DREAM_E_UNSUPPORTED, "tree shape out of range");
  *T = ts.T;
  return DREAM_OK;
}

extern "C" dream_status dream_tree_from_parents(const int32_t *parent, int32_t n_nodes, int32_t *depth, uint32_t *mask) {
  if (!parent || !depth || !mask) return fail(nullptr, DREAM_E_ARG, "null argument");
  if (n_nodes < 1 || n_nodes > 128) return fail(nullptr, DREAM_E_ARG, "n_nodes outside 1..128");
  if (parent[0] != -1) return fail(nullptr, DREAM_E_ARG, "node 0 is the root: parent[0] must be -1");
  for (int i = 0; i < n_nodes; ++i) {
    uint32_t *m = mask + 4 * i;
    if (i == 0) { depth[0] = 0; m[0] = m[1] = m[2] = m[3] = 0u; }
    else {
      int p = parent[i];
      if (p < 0 || p >= i) return fail(nullptr, DREAM_E_ARG, "parent[%d] = %d: parents precede their children", i, p);
      depth[i] = depth[p] + 1;
      for (int w = 0; w < 4; ++w) m[w] = mask[4 * p + w];
    }
    m[i >> 5] |= 1u << (i & 31);
  }
  return DREAM_OK;
}

static int ilog2(int v) { int s = 0; while ((1 << s) < v) ++s; return s; }
static int imax(int a, int b) { return a > b ? a : b; }
static int imin(int a, int b) { return a < b ? a : b; }

// Most rows one sequence contributes to any launch set: a verify takes T rows, the first draft pass
// D + 2 (root plus catch-up rows), a later pass its beam.
static int rows_per_seq_max(const TreeShape *ts) {
  int m = imax(ts->T, ts->D + 2);
  for (int p = 0; p <= ts->D; ++p) m = imax(m, ts->beam[p]);
  return m;
}

static dream_status check_config(const dream_config *c, TreeShape *ts) {
  if (!c) return fail(nullptr, DREAM_E_ARG, "null config");
  if (c->dtype != DREAM_F32 && c->dtype != DREAM_BF16) return fail(nullptr, DREAM_E_ARG, "dtype");
  if (c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256)
    return fail(nullptr, DREAM_E_UNSUPPORTED, "head_dim must be 64, 128 or 256");
  if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->n_kv_heads < 1 ||
      c->n_heads % c->n_kv_heads || c->d_ff < 8 || c->vocab < 2)
    return fail(nullptr, DREAM_E_ARG, "model shape");
  if (c->d_model % 8 || c->d_ff % 8) return fail(nullptr, DREAM_E_UNSUPPORTED, "d_model, d_ff must be multiples of 8");
  if (c->d_model > 16384) return fail(nullptr, DREAM_E_UNSUPPORTED, "d_model above 16384");
  if (c->vocab > TOPK_THREADS * TOPK_COLS) return fail(nullptr, DREAM_E_UNSUPPORTED, "vocab above 1048576");
  if (c->dtype == DREAM_BF16 && (c->d_model % 64 || c->d_ff % 64 || (c->n_heads * c->head_dim) % 64 || c->vocab % 8))
    return fail(nullptr, DREAM_E_UNSUPPORTED, "bf16: d_model, d_ff, n_heads*head_dim must be multiples of 64 and vocab of 8");
  if (c->dtype == DREAM_BF16 && 64 % (c->n_heads / c->n_kv_heads))
    return fail(nullptr, DREAM_E_UNSUPPORTED, "bf16: query heads per KV head must divide 64");
  if (c->max_batch < 1 || c->max_batch > DREAM_MAX_BATCH) return fail(nullptr, DREAM_E_ARG, "max_batch in 1..8");
  if (c->page_tokens < 16 || c->page_tokens > 256 || (c->page_tokens & (c->page_tokens - 1)))
    return fail(nullptr, DREAM_E_ARG, "page_tokens must be a power of two in 16..256");
  if (c->max_prompt < 1 || c->max_visual < 0 || c->max_visual > c->max_prompt || c->max_seq < c->max_prompt)
    return fail(nullptr, DREAM_E_ARG, "max_seq >= max_prompt >= max_visual required");
  if (tree_shape(c, ts)) return fail(nullptr, DREAM_E_UNSUPPORTED, "tree: depth<=15, topk<=16, beam*topk<=256, input nodes<=64, nodes<=128");
  if (c->max_batch * rows_per_seq_max(ts) > ROW_CHUNK)
    return fail(nullptr, DREAM_E_UNSUPPORTED, "max_batch * max(tree nodes, depth + 2, widest beam) must be <= 256");
  {   // the top-k kernel's last block merges at most 1024 candidates (vocabulary blocks x list length)
    int nv = (c->vocab + 1023) / 1024 * TOPK_MAX <= 1024 ? 4 : 16;
    int nsplit = (c->vocab + nv * TOPK_THREADS - 1) / (nv * TOPK_THREADS);
    if (nsplit * imax(ts->K, 2) > 1024)
      return fail(nullptr, DREAM_E_UNSUPPORTED, "vocab / 4096 * max(tree_topk, 2) must be <= 1024");
  }
  if (c->tap_mode == DREAM_TAP_FIXED) {
    if (c->tap_layer < 1 || c->tap_layer > c->n_layers) return fail(nullptr, DREAM_E_ARG, "tap_layer");
  } else if (c->tap_mode == DREAM_TAP_ENTROPY_MIN || c->tap_mode == DREAM_TAP_ENTROPY_MAX) {
    if (c->tap_lo < 1 || c->tap_hi > c->n_layers || c->tap_lo > c->tap_hi) return fail(nullptr, DREAM_E_ARG, "tap range");
  } else return fail(nullptr, DREAM_E_ARG, "tap_mode");
  if (c->draft_blocks != 0 && c->draft_blocks != 1 && c->draft_blocks != 3)
    return fail(nullptr, DREAM_E_ARG, "draft_blocks must be 1 (or 0) or 3");
  if (c->track_entropy != 0 && c->track_entropy != 1) return fail(nullptr, DREAM_E_ARG, "track_entropy must be 0 or 1");
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- arena

struct Carver {
  char *base;
  size_t off;
  template <typename U> U *take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    U *p = base ? reinterpret_cast<U *>(base + off) : nullptr;
    off += count * sizeof(U);
    return p;
  }
  void *take_bytes(size_t bytes) { return take<char>(bytes); }
};

static void derive(dream_ctx *c) {
  const dream_config &f = c->cfg;
  c->T = c->ts.T;
  c->esz = f.dtype == DREAM_BF16 ? 2 : 4;
  c->Hhd = f.n_heads * f.head_dim;
  c->kvN = 2 * f.n_kv_heads * f.head_dim;
  c->qkvN = c->Hhd + c->kvN;
  c->n_cand = f.tap_mode == DREAM_TAP_FIXED ? 1 : f.tap_hi - f.tap_lo + 1;
  c->tap_lo_eff = f.tap_mode == DREAM_TAP_FIXED ? f.tap_layer : f.tap_lo;
  c->cap_rows = f.max_seq + c->ts.NI;
  c->pps = (f.max_seq + f.page_tokens - 1) / f.page_tokens;
  c->n_pages = c->pps * f.max_batch;
  c->chunk = f.dtype == DREAM_BF16 ? TC_ROWS_SPLIT_1MMA : ROW_CHUNK;
  c->RM = (imax(ROW_CHUNK, f.max_prompt) + 15) & ~15;
  c->XR = c->RM;
  c->three = f.draft_blocks == 3;
}

static size_t carve(dream_ctx *c, char *base) {
  const dream_config &f = c->cfg;
  Carver a{base, 0};
  size_t e = c->esz;
  int MB = f.max_batch, NI = c->ts.NI, NC = c->ts.NC, T = c->T, d = f.d_model;
  c->kv_stride = (long long)c->n_pages * f.n_kv_heads * f.page_tokens * f.head_dim;
  c->layer_stride = 2 * c->kv_stride;
  c->kv_pool = a.take_bytes((size_t)f.n_layers * c->layer_stride * e);
  c->page_table = a.take<int>((size_t)MB * c->pps);
  c->status = a.take<int>(64);
  int *st = a.take<int>((size_t)MB * (9 + 3 * (DREAM_MAX_DEPTH + 1)));
  if (base) {
    c->sd.P = st; c->sd.pending = st + MB; c->sd.tap = st + 2 * MB; c->sd.nperm_d = st + 3 * MB;
    c->sd.nperm_m = st + 4 * MB; c->sd.n_new = st + 5 * MB; c->sd.last_P = st + 6 * MB;
    c->sd.last_A = st + 7 * MB;
    c->sd.new_tok = st + 9 * MB; c->sd.new_pos = c->sd.new_tok + MB * (DREAM_MAX_DEPTH + 1);
    c->sd.path = c->sd.new_pos + MB * (DREAM_MAX_DEPTH + 1);
  }
  size_t flat = (size_t)MB * 2 * f.n_kv_heads * c->cap_rows * f.head_dim;
  c->dself = a.take<float>(flat);
  c->dmem = a.take<float>(flat);
  c->dself2 = c->three ? a.take<float>(flat) : nullptr;
  c->dt.in_tok = a.take<int>((size_t)MB * NI); c->dt.in_depth = a.take<int>((size_t)MB * NI);
  c->dt.in_cand = a.take<int>((size_t)MB * NI); c->dt.in_cum = a.take<float>((size_t)MB * NI);
  c->dt.in_anc = a.take<unsigned long long>((size_t)MB * NI);
  c->dt.cand_tok = a.take<int>((size_t)MB * NC); c->dt.cand_par = a.take<int>((size_t)MB * NC);
  c->dt.cand_depth = a.take<int>((size_t)MB * NC); c->dt.cand_cum = a.take<float>((size_t)MB * NC);
  for (int b = 0; b < DREAM_MAX_BATCH; ++b) {
    if (b < MB) {
      c->itree[b].tokens = a.take<int>(T); c->itree[b].parent = a.take<int>(T);
      c->itree[b].depth = a.take<int>(T); c->itree[b].mask = a.take<uint32_t>(4 * T);
      c->itree[b].cum = a.take<float>(T);
    } else memset(&c->itree[b], 0, sizeof(TreePtrs));
  }
  for (int i = 0; i < 2; ++i) {
    c->rm[i].seq = a.take<int>(c->RM); c->rm[i].tok = a.take<int>(c->RM); c->rm[i].pos = a.take<int>(c->RM);
    c->rm[i].slot = a.take<int>(c->RM); c->rm[i].dst = a.take<int>(c->RM); c->rm[i].in = a.take<int>(c->RM);
    c->rm[i].vis_d = a.take<int>(c->RM); c->rm[i].vis_m = a.take<int>(c->RM);
  }
  c->gather_idx = a.take<int>(c->RM);
  c->ctx_pos = a.take<int>(f.max_prompt);
  c->flags = a.take<int>(f.max_prompt);
  c->vmask = a.take<uint32_t>((size_t)ROW_CHUNK * 4);
  c->x = a.take<float>((size_t)c->XR * d);
  c->x0 = a.take<float>((size_t)f.max_prompt * d);
  c->qbuf = a.take<float>((size_t)c->XR * c->Hhd);
  int planes = f.dtype == DREAM_BF16 ? 2 : 1;      // bf16 GEMM inputs: a high and a low row per token
  // attention outputs: whole prefill chunks of ROW_CHUNK rows
  c->attn_out = a.take_bytes((size_t)planes * ((c->XR + ROW_CHUNK - 1) / ROW_CHUNK * ROW_CHUNK) * c->Hhd * e);
  c->xn = a.take_bytes((size_t)planes * ROW_CHUNK * d * e);
  c->raw = a.take_bytes((size_t)planes * ROW_CHUNK * d * e);
  c->act = a.take_bytes((size_t)planes * ROW_CHUNK * f.d_ff * e);
  int lm_rows = ((imax(MB * T, MB * imax(c->ts.D + 2, f.tree_beam)) + 15) / 16) * 16;
  c->gemm_rows_lm = lm_rows;
  // GEMM output: the widest of every projection's footprint.  fp32: rows x N.  bf16: one region
  // per 64-row chunk, each with room for the stream-K partial-sum slots (bound for <= 192 SMs).
  {
    const int shapes[8][2] = {{c->qkvN, d}, {d, c->Hhd}, {2 * f.d_ff, d}, {d, f.d_ff}, {c->Hhd, d}, {c->kvN, d}, {f.vocab, d}, {0, 0}};
    size_t need = 0;
    for (int i = 0; shapes[i][0]; ++i) {
      int N = shapes[i][0], K = shapes[i][1];
      size_t fl;
      if (f.dtype == DREAM_BF16) {
        long long per = (gemm_tc_out_floats(192, TC_ROWS_SPLIT_1MMA, N, K) + 63) & ~63LL;
        long long per2 = (gemm_tc_out_floats(192, TC_ROWS_MAX, N, K) + 63) & ~63LL;
        fl = (size_t)imax(1, ROW_CHUNK / TC_ROWS_SPLIT_1MMA) * per;
        size_t fl2 = (size_t)imax(1, ROW_CHUNK / TC_ROWS_MAX) * per2;
        if (fl2 > fl) fl = fl2;
        size_t fl3 = (size_t)((gemm_tc_out_floats(192, ROW_CHUNK, N, K) + 63) & ~63LL);
        if (fl3 > fl) fl = fl3;
      } else fl = (size_t)ROW_CHUNK * N;
      if (fl > need) need = fl;
    }
    c->gout_floats = need;
  }
  c->gout = a.take<float>(c->gout_floats);
  c->rope_inv = a.take<double>(f.head_dim / 2);
  c->rope_tab = a.take<float2>((size_t)ROW_CHUNK * (f.head_dim / 2));
  c->lse_pre = a.take<float>((size_t)f.n_heads * f.max_prompt);
  c->ent_pre = a.take<float>((size_t)f.n_heads * f.max_prompt);
  c->ae = a.take<float>(f.n_layers);
  c->scores_all = a.take<float>((size_t)c->n_cand * imax(f.max_visual, 1));
  c->taps_store = a.take<float>((size_t)c->n_cand * f.max_prompt * d);
  c->tapbuf = a.take<float>((size_t)ROW_CHUNK * d);
  c->top_val = a.take<float>((size_t)ROW_CHUNK * TOPK_MAX);
  c->top_id = a.take<int>((size_t)ROW_CHUNK * TOPK_MAX);
  c->lse_rows = a.take<float>(ROW_CHUNK);
  c->am_rt_max = (rows_per_seq_max(&c->ts) * (f.n_heads / f.n_kv_heads) + AM_ROWS - 1) / AM_ROWS;
  if (f.dtype == DREAM_BF16) {
    size_t prow = (size_t)MB * AM_MAX_CHUNKS * f.n_kv_heads * c->am_rt_max * AM_ROWS;
    c->am_part_o = a.take<float>(prow * f.head_dim);
    c->am_part_ml = a.take<float>(prow * 2);
    c->am_part_u = f.track_entropy ? a.take<float>(prow) : nullptr;
  } else { c->am_part_o = nullptr; c->am_part_ml = nullptr; c->am_part_u = nullptr; }
  c->row_ent = f.track_entropy ? a.take<float>((size_t)f.n_layers * ROW_CHUNK * f.n_heads) : nullptr;
  c->ent_sum = f.track_entropy ? a.take<float>((size_t)MB * f.n_layers) : nullptr;
  // small blocks (1024 columns) while the merge of the blocks' lists stays within 1024 candidates
  c->tk_nv = (f.vocab + 1023) / 1024 * TOPK_MAX <= 1024 ? 4 : 16;
  c->tk_nsplit = (f.vocab + c->tk_nv * TOPK_THREADS - 1) / (c->tk_nv * TOPK_THREADS);
  c->tks.pv = a.take<float>((size_t)ROW_CHUNK * c->tk_nsplit * TOPK_MAX);
  c->tks.pi = a.take<int>((size_t)ROW_CHUNK * c->tk_nsplit * TOPK_MAX);
  c->tks.pm = a.take<float>((size_t)ROW_CHUNK * c->tk_nsplit);
  c->tks.pz = a.take<float>((size_t)ROW_CHUNK * c->tk_nsplit);
  c->tks.counter = a.take<int>(ROW_CHUNK);
  c->argmax_i = a.take<int>(ROW_CHUNK);
  c->margin_i = a.take<float>(ROW_CHUNK);
  c->accept_len_i = a.take<int>(MB);
  c->out_tokens_i = a.take<int>((size_t)MB * (DREAM_MAX_DEPTH + 1));
  c->comp_src_i = a.take<int>((size_t)MB * (DREAM_MAX_DEPTH + 1));
  return (a.off + 255) & ~(size_t)255;
}

extern "C" dream_status dream_arena_bytes(const dream_config *cfg, size_t *bytes) {
  if (!cfg || !bytes) return fail(nullptr, DREAM_E_ARG, "null argument");
  dream_ctx tmp;
  dream_status s = check_config(cfg, &tmp.ts);
  if (s) return s;
  tmp.cfg = *cfg;
  derive(&tmp);
  *bytes = carve(&tmp, nullptr);
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- GEMM dispatch

// How the rows of a bf16 GEMM input buffer are laid out for a launch set of R rows: up to 64 rows
// high and low rows alternate; more rows use two planes (high parts first, low parts lo_rows rows
// further on); up to 256 rows go through a GEMM in one launch (two token tiles per weight panel).
struct XMode { int mode, lo_rows; };
static XMode xmode(const dream_ctx *c, int R) {
  if (c->cfg.dtype != DREAM_BF16) return XMode{TC_X_PLAIN, 0};
  if (R <= TC_ROWS_SPLIT_1MMA) return XMode{TC_X_INTERLEAVED, 0};
  return XMode{TC_X_PLANAR, R <= TC_ROWS_MAX ? TC_ROWS_MAX : ROW_CHUNK};
}
static XLayout xlay(XMode m, long long width) {
  if (m.mode == TC_X_INTERLEAVED) return XLayout{2 * width, width};
  if (m.mode == TC_X_PLANAR) return XLayout{width, (long long)m.lo_rows * width};
  return XLayout{width, 0};
}

// out[r][c] = sum_k X[r][k] W[c][k] for r < rows, c < N; X holds the rows in layout m.
// Returns the descriptor consumers read the result through.
template <typename T>
static GemmOut gemm(dream_ctx *c, const void *W, const void *X, XMode m, int rows, int N, int K) {
  GemmOut g;
  if (sizeof(T) == 2) {
    // rows per launch: 64 (interleaved), 128 (two planes), 256 (two planes with room for two token tiles)
    int chunk = m.mode == TC_X_INTERLEAVED ? TC_ROWS_SPLIT_1MMA : (m.mode == TC_X_PLANAR && m.lo_rows >= 2 * TC_ROWS_MAX ? 2 * TC_ROWS_MAX : TC_ROWS_MAX);
    int nch = (rows + chunk - 1) / chunk;
    int slot_rows = nch > 1 ? chunk : rows;
    long long per = (gemm_tc_out_floats(c->tc.n_sms, slot_rows, N, K) + 63) & ~63LL;
    XLayout lay = xlay(m, K);
    for (int ch = 0; ch < nch; ++ch) {
      int rows_c = imin(chunk, rows - ch * chunk);
      const bf16 *Xc = (const bf16 *)X + (long long)ch * chunk * lay.row_stride;
      bool timed = c->prof_on && 2 * (c->prof_n + 1) <= (int)c->prof_ev.size();
      if (timed) cudaEventRecord(c->prof_ev[2 * c->prof_n], c->stream);
      if (!gemm_tc_launch(&c->tc, c->stream, W, Xc, m.mode, m.lo_rows, rows_c, slot_rows, N, K, c->gout + (long long)ch * per,
                          (long long)c->gout_floats - (long long)ch * per, &g))
        c->gemm_failed = 1;
      if (timed) { cudaEventRecord(c->prof_ev[2 * c->prof_n + 1], c->stream); c->prof_n++; c->prof_bytes += 2.0 * N * K; }
      c->launches++;
      c->tc_launches++;
    }
    g.base = c->gout; g.chunk_stride = per; g.chunk_shift = chunk == 64 ? 6 : (chunk == 128 ? 7 : 8);
    return g;
  }
  c->simt_launches++;
  dim3 grid((N + SG_BN - 1) / SG_BN, (rows + SG_BM - 1) / SG_BM);
  LAUNCH(c, (k_gemm_simt<T>), grid, 256, 0, (const T *)X, (const T *)W, c->gout, rows, N, K, N);
  g.base = c->gout; g.slot_stride = 0; g.chunk_stride = 0; g.chunk_shift = 30; g.ld = N; g.kb = 0; g.upc = 0;
  return g;
}

static PagedKV paged(dream_ctx *c, int layer) {
  PagedKV kv;
  kv.base = (char *)c->kv_pool + (size_t)layer * c->layer_stride * c->esz;
  kv.kv_stride = c->kv_stride;
  kv.page_table = c->page_table;
  kv.pages_per_seq = c->pps;
  kv.page_tokens = c->cfg.page_tokens;
  kv.page_shift = ilog2(c->cfg.page_tokens);
  kv.hkv = c->cfg.n_kv_heads;
  kv.hd = c->cfg.head_dim;
  return kv;
}
static FlatKV flat(dream_ctx *c, float *base) {
  FlatKV kv;
  kv.base = base; kv.cap = c->cap_rows; kv.hkv = c->cfg.n_kv_heads; kv.hd = c->cfg.head_dim;
  kv.split = c->cfg.dtype == DREAM_BF16 ? 1 : 0;
  return kv;
}
static const GemmOut NO_GEMM = {nullptr, 0, 0, 30, 0, 0, 0};

// ------------------------------------------------------------------------------------- prefix bounds

static int key_ub_of(const dream_ctx *c, int seq) { return c->key_ub0[seq] + (c->p_ub[seq] - c->n_prompt[seq]); }

// After an accept was enqueued: copy the device's verified lengths to a free pinned slot.
static void snapshot_lengths(dream_ctx *c) {
  int slot = -1;
  for (int i = 0; i < SNAP_SLOTS; ++i) {
    if (c->snap_busy[i] && cudaEventQuery(c->snap_ev[i]) == cudaSuccess) c->snap_busy[i] = 2;   // complete, still unread or read
    if (c->snap_busy[i] != 1 && (slot < 0 || c->snap_order[i] < c->snap_order[slot])) slot = i;
  }
  if (slot < 0) return;                                  // every slot still in flight: skip this one
  if (cudaMemcpyAsync(c->h_snap + slot * DREAM_MAX_BATCH, c->sd.P, sizeof(int) * c->cfg.max_batch, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaEventRecord(c->snap_ev[slot], c->stream) != cudaSuccess) { cudaGetLastError(); c->snap_busy[slot] = 0; return; }
  c->snap_busy[slot] = 1;
  c->snap_order[slot] = ++c->snap_clock;
  for (int b = 0; b < DREAM_MAX_BATCH; ++b) { c->snap_accepts[slot][b] = c->accepts[b]; c->snap_epoch[slot][b] = c->epoch[b]; }
}

// Before launches are planned: adopt the newest completed snapshot.  For a sequence that had k
// accepts enqueued after the snapshot the bound is its P then plus k (D + 1).
static void refresh_bounds(dream_ctx *c) {
  int best = -1;
  for (int i = 0; i < SNAP_SLOTS; ++i) {
    if (c->snap_busy[i] == 1 && cudaEventQuery(c->snap_ev[i]) == cudaSuccess) c->snap_busy[i] = 2;
    if (c->snap_busy[i] == 2 && (best < 0 || c->snap_order[i] > c->snap_order[best])) best = i;
  }
  cudaGetLastError();                                    // cudaErrorNotReady is not an error here
  if (best < 0) return;
  for (int b = 0; b < c->cfg.max_batch; ++b) {
    if (c->snap_epoch[best][b] != c->epoch[b] || c->phase[b] < PH_READY) continue;
    long long ub = (long long)c->h_snap[best * DREAM_MAX_BATCH + b] + (c->accepts[b] - c->snap_accepts[best][b]) * (c->ts.D + 1);
    if (ub < c->p_ub[b]) c->p_ub[b] = (int)ub;
  }
}

// ------------------------------------------------------------------------------------- init / free

template <int HD>
static const char *attn_tc_setup_all() {
  const char *w = attn_tc_setup<HD, false>();
  if (!w) w = attn_tc_setup<HD, true>();
  return w ? w : colsum_tc_setup<HD>();
}

static void free_host_side(dream_ctx *c) {
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  for (int i = 0; i < SNAP_SLOTS; ++i) if (c->snap_ev[i]) cudaEventDestroy(c->snap_ev[i]);
  cudaFreeHost(c->h_snap);
  cudaFreeHost(c->h_stage);
  delete c;
}

extern "C" dream_status dream_init(const dream_config *cfg, const dream_target_weights *tw,
                                   const dream_draft_weights *dw, void *arena, size_t arena_bytes,
                                   void *cuda_stream, dream_ctx **out) {
  if (!cfg || !tw || !dw || !arena || !out) return fail(nullptr, DREAM_E_ARG, "null argument");
  TreeShape ts;
  dream_status s = check_config(cfg, &ts);
  if (s) return s;
  if ((uintptr_t)arena & 255) return fail(nullptr, DREAM_E_ARG, "arena must be 256-byte aligned");
  dream_ctx *c = new dream_ctx();
  c->cfg = *cfg; c->ts = ts;
  derive(c);
  size_t need = carve(c, nullptr);
  if (arena_bytes < need) { delete c; return fail(nullptr, DREAM_E_NOMEM, "arena needs %zu bytes, got %zu", need, arena_bytes); }
  c->arena = (char *)arena; c->arena_bytes = need;
  carve(c, c->arena);
  c->stream = (cudaStream_t)cuda_stream;
  c->embed = tw->embed; c->ln_f = tw->ln_f; c->lm_head = tw->lm_head; c->dw = *dw;
  const void *dptr[] = {dw->ln1, dw->wqkv, dw->wo, dw->lnx, dw->xq, dw->xkv, dw->xo, dw->ln2, dw->wgu, dw->wd,
                        tw->embed, tw->ln_f, tw->lm_head};
  for (const void *p : dptr) if (!p) { delete c; return fail(nullptr, DREAM_E_ARG, "null weight pointer"); }
  if (c->three) {
    const void *d3[] = {dw->i_ln2, dw->i_wgu, dw->i_wd, dw->f_ln1, dw->f_wqkv, dw->f_wo, dw->f_ln2, dw->f_wgu, dw->f_wd};
    for (const void *p : d3) if (!p) { delete c; return fail(nullptr, DREAM_E_ARG, "draft_blocks = 3: null i_* or f_* weight pointer"); }
  }
  for (int l = 0; l < cfg->n_layers; ++l) {
    if (!tw->ln1[l] || !tw->wqkv[l] || !tw->wo[l] || !tw->ln2[l] || !tw->wgu[l] || !tw->wd[l]) {
      delete c; return fail(nullptr, DREAM_E_ARG, "null weight pointer in layer %d", l);
    }
    c->ln1.push_back(tw->ln1[l]); c->wqkv.push_back(tw->wqkv[l]); c->wo.push_back(tw->wo[l]);
    c->ln2.push_back(tw->ln2[l]); c->wgu.push_back(tw->wgu[l]); c->wd.push_back(tw->wd[l]);
  }
  cudaError_t e = cudaMemsetAsync(c->arena, 0, need, c->stream);
  if (e != cudaSuccess) { delete c; return fail(nullptr, DREAM_E_CUDA, "memset arena: %s", cudaGetErrorString(e)); }
  e = cudaHostAlloc((void **)&c->h_stage, sizeof(int) * ((size_t)cfg->max_batch * c->pps + 64 + cfg->max_batch * (DREAM_MAX_DEPTH + 2)), cudaHostAllocDefault);
  if (e != cudaSuccess) { delete c; return fail(nullptr, DREAM_E_CUDA, "pinned staging: %s", cudaGetErrorString(e)); }
  e = cudaHostAlloc((void **)&c->h_snap, sizeof(int) * SNAP_SLOTS * DREAM_MAX_BATCH, cudaHostAllocDefault);
  if (e != cudaSuccess) { cudaFreeHost(c->h_stage); delete c; return fail(nullptr, DREAM_E_CUDA, "pinned snapshots: %s", cudaGetErrorString(e)); }
  for (int i = 0; i < SNAP_SLOTS; ++i) {
    c->snap_busy[i] = 0; c->snap_order[i] = 0; c->snap_ev[i] = nullptr;
    if (cudaEventCreateWithFlags(&c->snap_ev[i], cudaEventDisableTiming) != cudaSuccess) {
      for (int j = 0; j < i; ++j) cudaEventDestroy(c->snap_ev[j]);
      cudaFreeHost(c->h_snap); cudaFreeHost(c->h_stage); delete c;
      return fail(nullptr, DREAM_E_CUDA, "cannot create an event");
    }
  }
  c->snap_clock = 0; c->last_verify_n = 0;
  for (int b = 0; b < DREAM_MAX_BATCH; ++b) { c->accepts[b] = 0; c->epoch[b] = 0; c->key_ub0[b] = 0; c->p_ub[b] = 0; c->n_prompt[b] = 0; }
  for (int p = c->n_pages - 1; p >= 0; --p) c->free_pages.push_back(p);
  for (int b = 0; b < DREAM_MAX_BATCH; ++b) c->phase[b] = PH_EMPTY;
  c->prefill_seq = -1;
  c->launches = 0; c->tc_launches = 0; c->simt_launches = 0; c->gemm_failed = 0;
  c->launch_err = cudaSuccess; c->launch_err_name = "";
  c->prof_on = 0; c->prof_n = 0; c->prof_bytes = 0.0;
  c->err[0] = 0;
  const char *pdl = getenv("DREAM_PDL");              // "0" serialises every launch (debugging aid)
  c->use_pdl = !(pdl && !strcmp(pdl, "0"));
  c->use_tc = cfg->dtype == DREAM_BF16;
  if (c->use_tc) {
    const char *why = gemm_tc_plan_init(&c->tc, c->status, c->use_pdl);
    if (why) { free_host_side(c); return fail(nullptr, DREAM_E_CUDA, "tensor-core GEMM set-up: %s", why); }
  }
  if (c->use_tc) {
    const char *why = cfg->head_dim == 64 ? attn_tc_setup_all<64>() : cfg->head_dim == 128 ? attn_tc_setup_all<128>() : attn_tc_setup_all<256>();
    if (why) { free_host_side(c); return fail(nullptr, DREAM_E_CUDA, "%s", why); }
  }
  k_rope_table<<<(cfg->head_dim / 2 + 127) / 128, 128, 0, c->stream>>>(c->rope_inv, cfg->head_dim, cfg->rope_theta);
  if (cudaGetLastError() != cudaSuccess) { free_host_side(c); return fail(nullptr, DREAM_E_CUDA, "rotary table launch failed"); }
  *out = c;
  return DREAM_OK;
}

extern "C" void dream_free(dream_ctx *c) {
  if (!c) return;
  cudaStreamSynchronize(c->stream);
  free_host_side(c);
}

extern "C" const char *dream_last_error(const dream_ctx *c) { return c ? c->err : g_init_error; }
extern "C" int64_t dream_launch_count(const dream_ctx *c) { return c ? c->launches : 0; }

extern "C" dream_status dream_poll(dream_ctx *c) {
  if (!c) return DREAM_E_ARG;
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  int st = 0;
  CUDA_OK(c, cudaMemcpy(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st == DREAM_DEV_TIMEOUT) return fail(c, DREAM_E_DEVICE_TIMEOUT, "a bounded device-side wait expired");
  if (st == DREAM_DEV_BAD_INDEX) return fail(c, DREAM_E_STATE, "a kernel met an index or capacity out of range");
  return DREAM_OK;
}

static dream_status check_seq(dream_ctx *c, int seq) {
  if (!c) return DREAM_E_ARG;
  if (seq < 0 || seq >= c->cfg.max_batch) return fail(c, DREAM_E_ARG, "sequence id %d out of range", seq);
  return DREAM_OK;
}

extern "C" dream_status dream_seq_reset(dream_ctx *c, int32_t seq) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  for (int p : c->seq_pages[seq]) c->free_pages.push_back(p);
  c->seq_pages[seq].clear();
  c->phase[seq] = PH_EMPTY;
  c->epoch[seq]++;
  if (c->prefill_seq == seq) c->prefill_seq = -1;
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- small kernels

__global__ void k_iota_rows(RowMeta rm, int seq, int n) {
  kernel_entry(TR_k_iota_rows);
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  rm.seq[i] = seq; rm.pos[i] = i; rm.slot[i] = i; rm.dst[i] = i; rm.in[i] = -1;
}
__global__ void k_set_seq(SeqDev s, int seq, int P, const int *pending_src, int nd, int nm) {
  kernel_entry(TR_k_set_seq);
  if (threadIdx.x) return;
  if (P >= 0) s.P[seq] = P;
  if (pending_src) s.pending[seq] = *pending_src;
  if (nd >= 0) { s.nperm_d[seq] = nd; s.nperm_m[seq] = nm; s.n_new[seq] = 0; }
}
__global__ void k_set_int(int *p, int v) {
  kernel_entry(TR_k_set_int);
  if (!threadIdx.x) *p = v;
}
__global__ void k_first_token(const int *top_id, const float *top_val, int *tok, float *margin) {
  kernel_entry(TR_k_first_token);
  if (threadIdx.x) return;
  if (tok) *tok = top_id[0];
  if (margin) *margin = top_val[0] - top_val[1];
}
__global__ void k_argmax_out(const int *top_id, const float *top_val, int R, int *am, float *mg, int *am2) {
  kernel_entry(TR_k_argmax_out);
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  am[r] = top_id[2 * r];
  if (am2) am2[r] = top_id[2 * r];
  if (mg) mg[r] = top_val[2 * r] - top_val[2 * r + 1];
}
__global__ void k_copy_f32(const float *src, float *dst, int n) {
  kernel_entry(TR_k_copy_f32);
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[i];
}
// Debug read-back: block h copies n values from src + h * head_stride to dst + h * n.  split: the
// source holds n high parts then n low parts (a draft-cache row of a bf16 configuration).
template <typename T>
__global__ void k_read_row(const T *src, long long head_stride, float *dst, int n, int split) {
  const T *s = src + (long long)blockIdx.x * head_stride;
  for (int i = threadIdx.x; i < n; i += blockDim.x)
    dst[(long long)blockIdx.x * n + i] = to_f(s[i]) + (split ? to_f(s[n + i]) : 0.f);
}

// Elements between the attention outputs of consecutive prefill chunks (ROW_CHUNK rows each; bf16
// configurations keep a plane of high and a plane of low rows per chunk).
static long long prefill_chunk_stride(const dream_ctx *c) {
  return (long long)(c->cfg.dtype == DREAM_BF16 ? 2 : 1) * ROW_CHUNK * c->Hhd;
}
template <typename T, int HD> struct AttnLaunch {
  // The output rows are laid out per prefill chunk of ROW_CHUNK rows (the O projection's input).
  static void prefill(dream_ctx *c, int layer, int seq, int n) {
    if (sizeof(T) == 2) {
      // causal attention of the n prompt rows on the tensor cores: one CTA per (KV head, 64 entries)
      // walks all keys up to its last row; row log-sum-exp and entropy (Eq. 2) come out of the same pass
      AttnTcArgs a = {};
      a.mode = AT_PREFILL;
      a.n_keys = n; a.lay = xlay(xmode(c, ROW_CHUNK), c->Hhd);
      a.out_chunk_rows = ROW_CHUNK; a.out_chunk_stride = prefill_chunk_stride(c);
      a.lse = c->lse_pre; a.ent = c->ent_pre;
      c->cur_seq[0] = seq;
      tc(c, a, layer, nullptr, 1, n, 0, nullptr);
      return;
    }
    dim3 grid((n + ATT_WARPS * ATT_PF_ROWS - 1) / (ATT_WARPS * ATT_PF_ROWS), c->cfg.n_heads);
    const XMode m = xmode(c, ROW_CHUNK);
    LAUNCH(c, (k_attn_prefill<T, HD>), grid, ATT_WARPS * 32, 0, c->qbuf, paged(c, layer), seq, n, c->cfg.n_heads,
           1.f / sqrtf((float)HD), (T *)c->attn_out, xlay(m, c->Hhd), ROW_CHUNK, prefill_chunk_stride(c), c->lse_pre, c->ent_pre);
  }
  static void colsum(dream_ctx *c, int layer, int seq, int n, int vis_start, int v, float *score) {
    if (v == 0) return;
    // the per-head sums land in the entropy buffer, which is idle between this layer's entropy mean
    // and the next layer's attention ([H][n] floats, v <= n)
    if (sizeof(T) == 2) {
      // tensor cores: 128 keys of one head per CTA, the query rows stream past (colsum_tc.cuh)
      const dream_config &f = c->cfg;
      ColsumTcArgs a = {};
      a.seq = seq; a.n = n; a.H = f.n_heads; a.G = f.n_heads / f.n_kv_heads;
      a.vis_start = vis_start; a.v = v; a.include_self = f.score_include_self;
      a.key0 = vis_start & ~63;
      a.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
      a.lse = c->lse_pre; a.part = c->ent_pre; a.status = c->status;
      const PagedKV kv = paged(c, layer);
      a.page_table = kv.page_table; a.pages_per_seq = kv.pages_per_seq; a.page_tokens = kv.page_tokens; a.page_shift = kv.page_shift;
      a.hkv = f.n_kv_heads;
      CUtensorMap mq, mk;
      bool ok;
      {
        const unsigned long long dims[4] = {(unsigned long long)HD, 2ull, (unsigned long long)f.n_heads, (unsigned long long)c->XR};
        const unsigned long long st[3] = {(unsigned long long)HD * 2, (unsigned long long)HD * 4, (unsigned long long)f.n_heads * HD * 4};
        const unsigned box[4] = {64u, 1u, 1u, (unsigned)CsShape<HD>::NQ};
        ok = at_map(&c->tc, &c->at_maps, c->qbuf, 4, dims, st, box, &mq);
      }
      {
        const unsigned long long dims[2] = {(unsigned long long)HD, (unsigned long long)c->n_pages * f.n_kv_heads * f.page_tokens};
        const unsigned long long st[1] = {(unsigned long long)HD * 2};
        const unsigned box[2] = {64u, (unsigned)imin(64, f.page_tokens)};
        ok = ok && at_map(&c->tc, &c->at_maps, kv.base, 2, dims, st, box, &mk);
      }
      if (!ok) { c->gemm_failed = 1; return; }
      const int n_tiles = (vis_start + v - a.key0 + CS_KEYS - 1) / CS_KEYS;
      cudaError_t e = colsum_tc_launch<HD>(c->stream, c->use_pdl, mq, mk, a, n_tiles);
      if (e != cudaSuccess && c->launch_err == cudaSuccess) { c->launch_err = e; c->launch_err_name = "k_colsum_tc"; }
      c->launches++;
      LAUNCH(c, k_colsum_heads, (v + 255) / 256, 256, 0, (const float *)c->ent_pre, c->cfg.n_heads, v, score);
      return;
    }
    LAUNCH(c, (k_colsum<T, HD>), dim3((v + ATT_WARPS - 1) / ATT_WARPS, c->cfg.n_heads), ATT_WARPS * 32, 0, c->qbuf, paged(c, layer), seq, n,
           c->cfg.n_heads, 1.f / sqrtf((float)HD), c->lse_pre, vis_start, v, c->cfg.score_include_self, c->ent_pre);
    LAUNCH(c, k_colsum_heads, (v + 255) / 256, 256, 0, (const float *)c->ent_pre, c->cfg.n_heads, v, score);
  }
  // The tcgen05 attention (bf16 configurations): split-K plan, tensor maps, launch, merge of the chunks.
  // cache: null = the paged target cache of `layer`, else a flat draft cache.
  static void tc(dream_ctx *c, AttnTcArgs a, int layer, const float *cache, int B, int rows_per_seq, int key_ub, const int *row_in,
                 const int *row_vis = nullptr) {
    const dream_config &f = c->cfg;
    const bool flat_kv = cache != nullptr;
    const int GROUP = flat_kv ? AtShape<HD, true>::GROUP : AtShape<HD, false>::GROUP;
    for (int b = 0; b < DREAM_MAX_BATCH; ++b) a.slot_seq[b] = b < B ? c->cur_seq[b] : 0;
    a.H = f.n_heads; a.G = f.n_heads / f.n_kv_heads; a.rows_per_seq = rows_per_seq; a.row_in = row_in; a.row_vis = row_vis;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
    a.n_rt = (rows_per_seq * a.G + 63) / 64;
    const int nb_ub = imax(1, (key_ub + AT_KBLK - 1) / AT_KBLK);
    const int tiles = f.n_kv_heads * a.n_rt * B;
    // as many key chunks as keep the grid in one wave of resident CTAs, the blocks dealt out evenly
    // (a chunk walks its blocks GROUP at a time)
    const int per_sm = flat_kv ? AtShape<HD, true>::CTAS_PER_SM : AtShape<HD, false>::CTAS_PER_SM;
    const int want = imin(imin(AM_MAX_CHUNKS, nb_ub), imax(1, c->tc.n_sms * per_sm / tiles));
    a.blocks_per_chunk = (nb_ub + want - 1) / want;
    a.n_chunks = (nb_ub + a.blocks_per_chunk - 1) / a.blocks_per_chunk;
    (void)GROUP;
    // a CTA walks every key its rows see: prefill, and row sets wider than the partials were sized for
    if (a.mode == AT_PREFILL || a.n_rt > c->am_rt_max) { a.n_chunks = 1; a.blocks_per_chunk = 1 << 24; }
    a.part_o = c->am_part_o; a.part_ml = c->am_part_ml; a.out = c->attn_out; a.status = c->status;
    a.hkv = f.n_kv_heads;
    CUtensorMap mq, mk, mv;
    bool ok;
    {
      const unsigned long long dims[4] = {(unsigned long long)HD, 2ull, (unsigned long long)f.n_heads, (unsigned long long)c->XR};
      const unsigned long long st[3] = {(unsigned long long)HD * 2, (unsigned long long)HD * 4, (unsigned long long)f.n_heads * HD * 4};
      const unsigned box[4] = {64u, 2u, (unsigned)a.G, (unsigned)(64 / a.G)};
      ok = at_map(&c->tc, &c->at_maps, c->qbuf, 4, dims, st, box, &mq);
    }
    if (flat_kv) {
      const unsigned long long dims[3] = {(unsigned long long)HD, 2ull, (unsigned long long)f.max_batch * 2 * f.n_kv_heads * c->cap_rows};
      const unsigned long long st[2] = {(unsigned long long)HD * 2, (unsigned long long)HD * 4};
      const unsigned box[3] = {64u, 1u, 64u};
      ok = ok && at_map(&c->tc, &c->at_maps, cache, 3, dims, st, box, &mk);
      mv = mk;
      a.flat_rows_per_head = c->cap_rows;
    } else {
      const PagedKV kv = paged(c, layer);
      const unsigned long long dims[2] = {(unsigned long long)HD, (unsigned long long)c->n_pages * f.n_kv_heads * f.page_tokens};
      const unsigned long long st[1] = {(unsigned long long)HD * 2};
      const unsigned box[2] = {64u, (unsigned)imin(64, f.page_tokens)};
      ok = ok && at_map(&c->tc, &c->at_maps, kv.base, 2, dims, st, box, &mk);
      ok = ok && at_map(&c->tc, &c->at_maps, (const bf16 *)kv.base + kv.kv_stride, 2, dims, st, box, &mv);
      a.page_table = kv.page_table; a.pages_per_seq = kv.pages_per_seq; a.page_tokens = kv.page_tokens; a.page_shift = kv.page_shift;
    }
    if (!ok) { c->gemm_failed = 1; return; }
    cudaError_t e = flat_kv ? attn_tc_launch<HD, true>(c->stream, c->use_pdl, mq, mk, mv, a, B)
                            : attn_tc_launch<HD, false>(c->stream, c->use_pdl, mq, mk, mv, a, B);
    if (e != cudaSuccess && c->launch_err == cudaSuccess) { c->launch_err = e; c->launch_err_name = "k_attn_tc"; }
    c->launches++;
    if (a.n_chunks > 1) {
      AttnMergeArgs m = {};
      m.row_in = row_in; m.row_vis = row_vis; m.rows_per_seq = rows_per_seq; m.H = a.H; m.G = a.G; m.n_chunks = a.n_chunks; m.n_rt = a.n_rt;
      m.part_o = a.part_o; m.part_ml = a.part_ml; m.out = a.out; m.lay = a.lay;
      m.part_u = a.part_u; m.row_ent = a.row_ent;
      long long items = (long long)B * rows_per_seq * f.n_heads * (HD / 4);
      LAUNCH(c, (k_attn_combine<HD>), (unsigned)((items + 255) / 256), 256, 0, m, B * rows_per_seq);
    }
  }
  static void tree(dream_ctx *c, int layer, int R, XMode m, int B, int key_ub) {
    if (sizeof(T) == 2) {
      AttnTcArgs a = {};
      a.mode = AT_VERIFY;
      a.next_w.ptr = (const char *)c->wo[layer]; a.next_w.bytes = (unsigned long long)c->cfg.d_model * c->Hhd * 2;
      a.prefix_len = c->sd.P; a.mask = c->vmask; a.tail_len = c->T; a.lay = xlay(m, c->Hhd);
      if (c->row_ent) { a.row_ent = c->row_ent + (size_t)layer * ROW_CHUNK * c->cfg.n_heads; a.part_u = c->am_part_u; }
      tc(c, a, layer, nullptr, B, c->T, key_ub, nullptr);
      return;
    }
    dim3 grid((R + ATT_WARPS - 1) / ATT_WARPS, c->cfg.n_heads);
    if (c->row_ent)
      LAUNCH(c, (k_attn_tree<T, HD, true>), grid, ATT_WARPS * 32, 0, c->qbuf, paged(c, layer), c->rm[0].seq, c->rm[0].in,
             c->sd.P, c->vmask, R, c->T, c->cfg.n_heads, 1.f / sqrtf((float)HD), (T *)c->attn_out, xlay(m, c->Hhd),
             c->row_ent + (size_t)layer * ROW_CHUNK * c->cfg.n_heads);
    else
      LAUNCH(c, (k_attn_tree<T, HD, false>), grid, ATT_WARPS * 32, 0, c->qbuf, paged(c, layer), c->rm[0].seq, c->rm[0].in,
             c->sd.P, c->vmask, R, c->T, c->cfg.n_heads, 1.f / sqrtf((float)HD), (T *)c->attn_out, xlay(m, c->Hhd), (float *)nullptr);
  }
  // row_vis: null, or per row the number of leading cache rows a permanent row sees (RowMeta::vis_d / vis_m).
  // tail: false when no row of the launch reads the tree region (the draft's run over the context).
  static void draft(dream_ctx *c, const RowMeta &rm, float *cache, const int *nperm, int strict, int R, XMode m, int B,
                    int rows_per_seq, int key_ub, const int *row_vis = nullptr, bool tail = true) {
    if (sizeof(T) == 2) {
      AttnTcArgs a = {};
      a.mode = AT_DRAFT;
      a.prefix_len = nperm; a.anc = c->dt.in_anc; a.anc_stride = c->ts.NI; a.strict = strict; a.tail_len = tail ? c->ts.NI : 0;
      a.lay = xlay(m, c->Hhd);
      tc(c, a, 0, cache, B, rows_per_seq, key_ub, rm.in, row_vis);
      return;
    }
    dim3 grid((R + ATT_WARPS - 1) / ATT_WARPS, c->cfg.n_heads);
    LAUNCH(c, (k_attn_draft<T, HD>), grid, ATT_WARPS * 32, 0, c->qbuf, flat(c, cache), rm.seq, rm.in, row_vis, nperm,
           c->dt.in_anc, c->ts.NI, strict, R, c->cfg.n_heads, 1.f / sqrtf((float)HD), (T *)c->attn_out, xlay(m, c->Hhd));
  }
};

#define HD_DISPATCH(c, T, call)                                   \
  do {                                                            \
    if ((c)->cfg.head_dim == 64) AttnLaunch<T, 64>::call;         \
    else if ((c)->cfg.head_dim == 128) AttnLaunch<T, 128>::call;  \
    else AttnLaunch<T, 256>::call;                                \
  } while (0)

// x (+= GEMM output) -> RMSNorm -> GEMM input rows in c->xn; see k_resid_norm for the side outputs.
template <typename T>
static void norm_rows(dream_ctx *c, float *x, const GemmOut &gin, bool has_in, const void *gain, int rows, XMode m,
                      float *copy = nullptr, const int *row_seq = nullptr, const int *tap = nullptr, int layer = 0,
                      bool want_raw = false) {
  const int d4 = c->cfg.d_model / 4;
  int nv = 1;
  while ((d4 + nv - 1) / nv > 1024) nv *= 2;                 // d_model <= 16384 by check_config
  const int threads = ((d4 + nv - 1) / nv + 31) & ~31;
  if (nv == 1) LAUNCH(c, (k_resid_norm<T, 1>), rows, threads, 0, x, gin, has_in ? 1 : 0, (const T *)gain, c->cfg.rms_eps, c->cfg.d_model,
         (T *)c->xn, copy, row_seq, tap, layer, want_raw ? (T *)c->raw : (T *)nullptr, xlay(m, c->cfg.d_model));
  else if (nv == 2) LAUNCH(c, (k_resid_norm<T, 2>), rows, threads, 0, x, gin, has_in ? 1 : 0, (const T *)gain, c->cfg.rms_eps, c->cfg.d_model,
         (T *)c->xn, copy, row_seq, tap, layer, want_raw ? (T *)c->raw : (T *)nullptr, xlay(m, c->cfg.d_model));
  else LAUNCH(c, (k_resid_norm<T, 4>), rows, threads, 0, x, gin, has_in ? 1 : 0, (const T *)gain, c->cfg.rms_eps, c->cfg.d_model,
         (T *)c->xn, copy, row_seq, tap, layer, want_raw ? (T *)c->raw : (T *)nullptr, xlay(m, c->cfg.d_model));
}
template <typename T>
static GemmOut mlp_rows(dream_ctx *c, const void *wgu, const void *wd, int rows, XMode m) {
  const dream_config &f = c->cfg;
  GemmOut g = gemm<T>(c, wgu, c->xn, m, rows, 2 * f.d_ff, f.d_model);
  LAUNCH(c, (k_silu_mul<T>), dim3((f.d_ff + 1023) / 1024, rows), 256, 0, g, (T *)c->act, f.d_ff, xlay(m, f.d_ff));
  return gemm<T>(c, wd, c->act, m, rows, f.d_model, f.d_ff);
}

// ------------------------------------------------------------------------------------- prefill

template <typename T>
static dream_status prefill_impl(dream_ctx *c, int seq, const void *visual, int v, int vis_start,
                                 const int *ids, int q, int *first_token, float *first_margin,
                                 float *layer_entropy, int *tap_layer) {
  const dream_config &f = c->cfg;
  // The prompt goes through the projections ROW_CHUNK rows at a time: the weights stream once per
  // chunk (bf16: two token tiles of 128 rows share every weight panel).
  int n = q + v, d = f.d_model, L = f.n_layers, CH = ROW_CHUNK;
  LAUNCH(c, k_iota_rows, (n + 255) / 256, 256, 0, c->rm[0], seq, n);
  LAUNCH(c, (k_build_prompt<T>), n, 256, 0, (const T *)c->embed, (const T *)visual, ids, vis_start, v, c->x, c->x0,
         d, f.vocab, c->status);
  const XMode mp = xmode(c, CH);           // the layout of a full chunk of rows
  const XMode m1 = xmode(c, 1);
  const long long att_chunk = prefill_chunk_stride(c);
  for (int l = 0; l < L; ++l) {
    for (int r0 = 0; r0 < n; r0 += CH) {
      int rows = imin(CH, n - r0);
      norm_rows<T>(c, c->x + (size_t)r0 * d, NO_GEMM, false, c->ln1[l], rows, mp);
      GemmOut g = gemm<T>(c, c->wqkv[l], c->xn, mp, rows, c->qkvN, d);
      LAUNCH(c, (k_qkv_post_target<T>), dim3(rows, (c->qkvN / 8 + 255) / 256), 256, 0, g, c->rm[0].seq, c->rm[0].pos, c->rm[0].slot, r0, c->qbuf,
             paged(c, l), f.n_heads, c->rope_inv, (const float2 *)nullptr);
    }
    HD_DISPATCH(c, T, prefill(c, l, seq, n));
    LAUNCH(c, k_entropy_mean, 1, 1024, 0, c->ent_pre, f.n_heads * n, c->ae + l,
           c->ent_sum ? c->ent_sum + (size_t)seq * L + l : (float *)nullptr);
    int cand = l + 1 - c->tap_lo_eff;
    bool is_cand = cand >= 0 && cand < c->n_cand;
    if (is_cand) HD_DISPATCH(c, T, colsum(c, l, seq, n, vis_start, v, c->scores_all + (size_t)cand * imax(f.max_visual, 1)));
    for (int r0 = 0; r0 < n; r0 += CH) {
      int rows = imin(CH, n - r0);
      float *xr = c->x + (size_t)r0 * d;
      GemmOut g = gemm<T>(c, c->wo[l], (const T *)c->attn_out + (long long)(r0 / CH) * att_chunk, mp, rows, d, c->Hhd);
      norm_rows<T>(c, xr, g, true, c->ln2[l], rows, mp);
      g = mlp_rows<T>(c, c->wgu[l], c->wd[l], rows, mp);
      float *copy = is_cand ? c->taps_store + ((size_t)cand * f.max_prompt + r0) * d : nullptr;
      LAUNCH(c, k_resid_add, dim3(rows, (d + 1023) / 1024), 256, 0, xr, g, d, copy);
    }
  }
  // first token: LM head on the last prompt row
  norm_rows<T>(c, c->x + (size_t)(n - 1) * d, NO_GEMM, false, c->ln_f, 1, m1);
  GemmOut g = gemm<T>(c, c->lm_head, c->xn, m1, 1, f.vocab, d);
  TOPK_LAUNCH(c, dim3(1, c->tk_nsplit), g, f.vocab, 2, c->tk_nsplit, c->tks, c->top_val, c->top_id, c->lse_rows, (float *)nullptr);
  LAUNCH(c, k_first_token, 1, 32, 0, c->top_id, c->top_val, first_token, first_margin);
  LAUNCH(c, k_set_seq, 1, 32, 0, c->sd, seq, n, c->top_id, -1, -1);
  LAUNCH(c, k_select_tap, 1, 32, 0, c->ae, f.tap_mode, f.tap_layer, f.tap_lo, f.tap_hi, c->sd.tap + seq, tap_layer);
  if (layer_entropy) LAUNCH(c, k_copy_f32, (L + 255) / 256, 256, 0, c->ae, layer_entropy, L);
  return DREAM_OK;
}

extern "C" dream_status dream_prefill(dream_ctx *c, int32_t seq, const void *visual, int32_t v,
                                      int32_t vis_start, const int32_t *ids, int32_t q,
                                      int32_t *first_token, float *first_margin, float *layer_entropy,
                                      int32_t *tap_layer) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  const dream_config &f = c->cfg;
  if (v < 0 || q < 0 || v + q < 1 || (v && !visual) || (q && !ids)) return fail(c, DREAM_E_ARG, "prompt: need v + q >= 1 and buffers");
  if (vis_start < 0 || vis_start > q) return fail(c, DREAM_E_ARG, "vis_start must lie in [0, q]");
  if (v > f.max_visual || v + q > f.max_prompt) return fail(c, DREAM_E_CAPACITY, "prompt of %d (+%d visual) exceeds max_prompt/max_visual", v + q, v);
  if (c->phase[seq] != PH_EMPTY) return fail(c, DREAM_E_STATE, "sequence %d is live; dream_seq_reset it first", seq);
  if ((int)c->free_pages.size() < c->pps) return fail(c, DREAM_E_CAPACITY, "page pool exhausted");
  int *stage = c->h_stage + (size_t)seq * c->pps;
  for (int i = 0; i < c->pps; ++i) {
    int p = c->free_pages.back();
    c->free_pages.pop_back();
    c->seq_pages[seq].push_back(p);
    stage[i] = p;
  }
  CUDA_OK(c, cudaMemcpyAsync(c->page_table + (size_t)seq * c->pps, stage, sizeof(int) * c->pps, cudaMemcpyHostToDevice, c->stream));
  if (f.dtype == DREAM_BF16) s = prefill_impl<bf16>(c, seq, visual, v, vis_start, ids, q, first_token, first_margin, layer_entropy, tap_layer);
  else s = prefill_impl<float>(c, seq, visual, v, vis_start, ids, q, first_token, first_margin, layer_entropy, tap_layer);
  if (s) return s;
  s = call_done(c);
  if (s) return s;
  c->phase[seq] = PH_PREFILLED;
  c->n_prompt[seq] = v + q; c->p_ub[seq] = v + q; c->epoch[seq]++;
  c->prefill_seq = seq; c->pf_v = v; c->pf_vis_start = vis_start; c->pf_q = q;
  return DREAM_OK;
}

extern "C" dream_status dream_set_tap(dream_ctx *c, int32_t seq, int32_t tap_layer) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  if (c->phase[seq] != PH_PREFILLED || c->prefill_seq != seq) return fail(c, DREAM_E_STATE, "dream_set_tap follows dream_prefill of the same sequence");
  if (tap_layer < c->tap_lo_eff || tap_layer >= c->tap_lo_eff + c->n_cand)
    return fail(c, DREAM_E_ARG, "tap layer %d outside the stored range [%d, %d]", tap_layer, c->tap_lo_eff, c->tap_lo_eff + c->n_cand - 1);
  LAUNCH(c, k_set_int, 1, 32, 0, c->sd.tap + seq, tap_layer);
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- compression

// One pass of the draft over R rows whose inputs sit in c->x (Section 3.1; Section 4 for the three
// blocks): everything up to the last MLP's down projection, whose output (still to be added to c->x)
// is returned.  vis: the row set holds permanent rows (context or catch-up rows, RowMeta::vis_d/vis_m).
// tail: rows of the tree region exist.  context: the rows are the compressed context itself, which
// needs nothing behind the final block's K/V rows.
template <typename T>
static GemmOut draft_rows(dream_ctx *c, const RowMeta &rm, int R, XMode xm, int B, int m, int key_ub, bool vis, bool tail,
                          bool context, const float2 *rope_tab) {
  const dream_config &f = c->cfg;
  const int d = f.d_model;
  const dream_draft_weights &w = c->dw;
  const int *vd = vis ? rm.vis_d : nullptr, *vm = vis ? rm.vis_m : nullptr;
  GemmOut g;
  norm_rows<T>(c, c->x, NO_GEMM, false, w.ln1, R, xm);
  g = gemm<T>(c, w.wqkv, c->xn, xm, R, c->qkvN, d);
  LAUNCH(c, k_qkv_post_draft, dim3(R, (c->qkvN / 8 + 255) / 256), 256, 0, g, rm.seq, rm.pos, rm.dst, 0, 1, c->qbuf, flat(c, c->dself), f.n_heads, c->rope_inv, rope_tab);
  HD_DISPATCH(c, T, draft(c, rm, c->dself, c->sd.nperm_d, 0, R, xm, B, m, key_ub, vd, tail));
  g = gemm<T>(c, w.wo, c->attn_out, xm, R, d, c->Hhd);
  if (c->three) {
    norm_rows<T>(c, c->x, g, true, w.i_ln2, R, xm);
    g = mlp_rows<T>(c, w.i_wgu, w.i_wd, R, xm);
  }
  norm_rows<T>(c, c->x, g, true, w.lnx, R, xm);
  g = gemm<T>(c, w.xq, c->xn, xm, R, c->Hhd, d);
  LAUNCH(c, k_gemm_to_q, dim3(R, (c->Hhd + 1023) / 1024), 256, 0, g, c->qbuf, f.n_heads, f.head_dim, sizeof(T) == 2 ? 1 : 0);
  HD_DISPATCH(c, T, draft(c, rm, c->dmem, c->sd.nperm_m, 1, R, xm, B, m, key_ub, vm, tail));
  g = gemm<T>(c, w.xo, c->attn_out, xm, R, d, c->Hhd);
  norm_rows<T>(c, c->x, g, true, w.ln2, R, xm);
  g = mlp_rows<T>(c, w.wgu, w.wd, R, xm);
  if (c->three) {
    norm_rows<T>(c, c->x, g, true, w.f_ln1, R, xm);
    g = gemm<T>(c, w.f_wqkv, c->xn, xm, R, c->qkvN, d);
    LAUNCH(c, k_qkv_post_draft, dim3(R, (c->qkvN / 8 + 255) / 256), 256, 0, g, rm.seq, rm.pos, rm.dst, 0, 1, c->qbuf, flat(c, c->dself2), f.n_heads, c->rope_inv, rope_tab);
    if (context) return g;
    HD_DISPATCH(c, T, draft(c, rm, c->dself2, c->sd.nperm_d, 0, R, xm, B, m, key_ub, vd, tail));
    g = gemm<T>(c, w.f_wo, c->attn_out, xm, R, d, c->Hhd);
    norm_rows<T>(c, c->x, g, true, w.f_ln2, R, xm);
    g = mlp_rows<T>(c, w.f_wgu, w.f_wd, R, xm);
  }
  return g;
}

template <typename T>
static dream_status compress_impl(dream_ctx *c, int seq, int k, const int *forced, int *kept, float *scores) {
  const dream_config &f = c->cfg;
  int v = c->pf_v, q = c->pf_q, n = v + q, d = f.d_model, nc = q + k, CH = c->chunk;
  LAUNCH(c, k_select_visual, 1, 1024, 0, c->scores_all, (long long)imax(f.max_visual, 1), c->sd.tap + seq, c->tap_lo_eff,
         v, k, c->pf_vis_start, n, forced, kept, scores, c->ctx_pos, c->flags);
  // draft self-attention K/V of the compressed context, from the input embeddings
  const char *wkv = (const char *)c->dw.wqkv + (size_t)c->Hhd * d * c->esz;
  const XMode m1 = xmode(c, 1);
  for (int r0 = 0; r0 < nc && !c->three; r0 += CH) {
    int rows = imin(CH, nc - r0);
    LAUNCH(c, k_ctx_rows, (rows + 255) / 256, 256, 0, c->ctx_pos + r0, rows, 0, seq, c->rm[0], c->gather_idx, r0, 0);
    LAUNCH(c, (k_gather_rows<float>), rows, 256, 0, c->x0, c->gather_idx, c->x, d, (const int *)nullptr, 0, 0LL, XLayout{d, 0});
    norm_rows<T>(c, c->x, NO_GEMM, false, c->dw.ln1, rows, m1);
    GemmOut g = gemm<T>(c, wkv, c->xn, m1, rows, c->kvN, d);
    LAUNCH(c, k_qkv_post_draft, dim3(rows, (c->kvN / 8 + 255) / 256), 256, 0, g, c->rm[0].seq, c->rm[0].pos, c->rm[0].dst, 0, 0, (float *)nullptr,
           flat(c, c->dself), f.n_heads, c->rope_inv, (const float2 *)nullptr);
  }
  // cross-attention memory: tapped features at the context positions, projected (Eq. 1)
  int nm = f.xattn_full_memory ? n : nc;
  for (int r0 = 0; r0 < nm; r0 += CH) {
    int rows = imin(CH, nm - r0);
    LAUNCH(c, k_ctx_rows, (rows + 255) / 256, 256, 0, c->ctx_pos + r0, rows, f.xattn_full_memory, seq, c->rm[0], c->gather_idx, r0, 0);
    LAUNCH(c, (k_gather_rows<T>), rows, 256, 0, c->taps_store, c->gather_idx, (T *)c->raw, d, c->sd.tap + seq, c->tap_lo_eff,
           (long long)f.max_prompt * d, xlay(m1, d));
    GemmOut g = gemm<T>(c, c->dw.xkv, c->raw, m1, rows, c->kvN, d);
    LAUNCH(c, k_mem_append, dim3(rows, (c->kvN + 1023) / 1024), 256, 0, g, c->rm[0].seq, c->rm[0].dst, (const int *)nullptr, (const int *)nullptr, 0, flat(c, c->dmem));
  }
  LAUNCH(c, k_set_seq, 1, 32, 0, c->sd, seq, -1, (const int *)nullptr, nc, nm);
  if (c->three) {
    // The three-block draft runs over its compressed context (the memory above is complete by now):
    // a chunk of rows at a time, each row seeing the rows up to itself in the decoder blocks' caches
    // and the memory rows of earlier positions.  The cache rows behind a chunk are not written yet;
    // no row of the chunk sees them.
    c->cur_seq[0] = seq;
    for (int r0 = 0; r0 < nc; r0 += CH) {
      int rows = imin(CH, nc - r0);
      const XMode xm = xmode(c, rows);
      LAUNCH(c, k_ctx_rows, (rows + 255) / 256, 256, 0, c->ctx_pos + r0, rows, 0, seq, c->rm[0], c->gather_idx, r0, f.xattn_full_memory);
      LAUNCH(c, (k_gather_rows<float>), rows, 256, 0, c->x0, c->gather_idx, c->x, d, (const int *)nullptr, 0, 0LL, XLayout{d, 0});
      draft_rows<T>(c, c->rm[0], rows, xm, 1, rows, imax(nc, nm), true, false, true, (const float2 *)nullptr);
    }
  }
  return DREAM_OK;
}

extern "C" dream_status dream_compress_visual(dream_ctx *c, int32_t seq, int32_t k, const int32_t *forced,
                                              int32_t *kept, float *scores) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  if (c->phase[seq] != PH_PREFILLED || c->prefill_seq != seq)
    return fail(c, DREAM_E_STATE, "dream_compress_visual follows dream_prefill of the same sequence");
  if (k < 0 || k > c->pf_v) return fail(c, DREAM_E_ARG, "k = %d outside [0, v = %d]", k, c->pf_v);
  s = c->cfg.dtype == DREAM_BF16 ? compress_impl<bf16>(c, seq, k, forced, kept, scores)
                                 : compress_impl<float>(c, seq, k, forced, kept, scores);
  if (s) return s;
  s = call_done(c);
  if (s) return s;
  c->phase[seq] = PH_READY;
  c->key_ub0[seq] = c->pf_q + (c->cfg.xattn_full_memory ? c->pf_v : k);
  c->prefill_seq = -1;
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- batch helpers

static dream_status make_batch(dream_ctx *c, const int *seqs, int n_seqs, const dream_tree *trees, bool need_cum,
                               TreeBatch *tb) {
  if (!c) return DREAM_E_ARG;
  if (!seqs || n_seqs < 1 || n_seqs > c->cfg.max_batch) return fail(c, DREAM_E_ARG, "n_seqs outside 1..max_batch");
  memset(tb, 0, sizeof(*tb));
  for (int b = 0; b < n_seqs; ++b) {
    dream_status s = check_seq(c, seqs[b]);
    if (s) return s;
    for (int a = 0; a < b; ++a) if (seqs[a] == seqs[b]) return fail(c, DREAM_E_ARG, "sequence %d listed twice", seqs[b]);
    tb->seq[b] = seqs[b];
    if (trees) {
      const dream_tree &t = trees[b];
      if (!t.tokens || !t.parent || !t.depth || !t.mask) return fail(c, DREAM_E_ARG, "tree %d has a null buffer", b);
      tb->t[b].tokens = t.tokens; tb->t[b].parent = t.parent; tb->t[b].depth = t.depth;
      tb->t[b].mask = t.mask; tb->t[b].cum = t.cum_logp;
    } else tb->t[b] = c->itree[seqs[b]];
    (void)need_cum;
  }
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- draft

template <typename T>
static dream_status draft_impl(dream_ctx *c, const TreeBatch &tb, int B) {
  const dream_config &f = c->cfg;
  const TreeShape &ts = c->ts;
  int d = f.d_model, cur = 0;
  for (int b = 0; b < B; ++b) c->cur_seq[b] = tb.seq[b];
  int key_ub = 0;                 // most keys any listed sequence can hold in a draft cache
  for (int b = 0; b < B; ++b) key_ub = imax(key_ub, key_ub_of(c, tb.seq[b]) + ts.D + 1 + ts.NI);
  for (int p = 1; p <= ts.D; ++p) {
    int m = p == 1 ? ts.D + 2 : ts.beam[p - 1];
    int R = B * m;
    const XMode xm = xmode(c, R);
    RowMeta &rm = c->rm[cur], &rn = c->rm[cur ^ 1];
    if (p == 1) LAUNCH(c, k_draft_begin, 1, 32, 0, tb, B, c->sd, c->dt, ts, rm, m, c->cap_rows, c->status);
    LAUNCH(c, (k_embed<T>), dim3(R, (d + 1023) / 1024), 256, 0, (const T *)c->embed, rm.tok, c->x, d, f.vocab, c->status,
           (const int *)rm.pos, (const double *)c->rope_inv, c->rope_tab, f.head_dim / 2);
    // pass 1 of the three-block draft carries the catch-up rows through every block
    GemmOut g = draft_rows<T>(c, rm, R, xm, B, m, key_ub, c->three && p == 1, true, false, (const float2 *)c->rope_tab);
    // e^M = x: the raw copy feeds the memory projection, the normalised copy the LM head
    norm_rows<T>(c, c->x, g, true, c->ln_f, R, xm, nullptr, nullptr, nullptr, 0, true);
    if (p < ts.D) {     // the last pass's features have no descendants to attend to them
      g = gemm<T>(c, c->dw.xkv, c->raw, xm, R, c->kvN, d);
      LAUNCH(c, k_mem_append, dim3(R, (c->kvN + 1023) / 1024), 256, 0, g, rm.seq, rm.dst, rm.in, c->sd.nperm_m, 0, flat(c, c->dmem));
    }
    g = gemm<T>(c, c->lm_head, c->xn, xm, R, f.vocab, d);
    TOPK_LAUNCH(c, dim3(R, c->tk_nsplit), g, f.vocab, ts.K, c->tk_nsplit, c->tks, c->top_val, c->top_id, c->lse_rows, (float *)nullptr);
    int next_m = p < ts.D ? ts.beam[p] : 1;
    LAUNCH(c, k_tree_expand, B, 128, 0, tb, c->sd, c->dt, ts, p, m, c->top_val, c->top_id, c->lse_rows, rn, next_m);
    cur ^= 1;
  }
  LAUNCH(c, k_tree_finalize, B, 256, 2 * ts.NC * sizeof(int), tb, c->sd, c->dt, ts);
  return DREAM_OK;
}

extern "C" dream_status dream_draft_tree(dream_ctx *c, const int32_t *seqs, int32_t n_seqs, const dream_tree *trees) {
  TreeBatch tb;
  dream_status s = make_batch(c, seqs, n_seqs, trees, true, &tb);
  if (s) return s;
  for (int b = 0; b < n_seqs; ++b)
    if (c->phase[seqs[b]] != PH_READY) return fail(c, DREAM_E_STATE, "sequence %d: dream_draft_tree follows dream_compress_visual or dream_accept", seqs[b]);
  refresh_bounds(c);
  s = c->cfg.dtype == DREAM_BF16 ? draft_impl<bf16>(c, tb, n_seqs) : draft_impl<float>(c, tb, n_seqs);
  if (s) return s;
  s = call_done(c);
  if (s) return s;
  for (int b = 0; b < n_seqs; ++b) c->phase[seqs[b]] = PH_DRAFTED;
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- verify

template <typename T>
static dream_status verify_impl(dream_ctx *c, const TreeBatch &tb, int B, int *argmax, float *margin, float *logits) {
  const dream_config &f = c->cfg;
  int d = f.d_model, L = f.n_layers, R = B * c->T;
  const XMode xm = xmode(c, R);
  RowMeta &rm = c->rm[0];
  int key_ub = 0;
  for (int b = 0; b < B; ++b) { key_ub = imax(key_ub, c->p_ub[tb.seq[b]] + c->T); c->cur_seq[b] = tb.seq[b]; }
  LAUNCH(c, k_verify_setup, (R + 127) / 128, 128, 0, tb, B, c->T, c->sd, rm, c->vmask, f.max_seq, c->status);
  LAUNCH(c, (k_embed<T>), dim3(R, (d + 1023) / 1024), 256, 0, (const T *)c->embed, rm.tok, c->x, d, f.vocab, c->status,
           (const int *)rm.pos, (const double *)c->rope_inv, c->rope_tab, f.head_dim / 2);
  GemmOut gd = NO_GEMM, g;
  for (int l = 0; l < L; ++l) {
    // the first norm completes S^l (for l >= 1) and captures it where a sequence taps layer l
    norm_rows<T>(c, c->x, gd, l > 0, c->ln1[l], R, xm, l > 0 ? c->tapbuf : nullptr, rm.seq, c->sd.tap, l);
    g = gemm<T>(c, c->wqkv[l], c->xn, xm, R, c->qkvN, d);
    LAUNCH(c, (k_qkv_post_target<T>), dim3(R, (c->qkvN / 8 + 255) / 256), 256, 0, g, rm.seq, rm.pos, rm.slot, 0, c->qbuf, paged(c, l), f.n_heads, c->rope_inv, (const float2 *)c->rope_tab);
    HD_DISPATCH(c, T, tree(c, l, R, xm, B, key_ub));
    g = gemm<T>(c, c->wo[l], c->attn_out, xm, R, d, c->Hhd);
    norm_rows<T>(c, c->x, g, true, c->ln2[l], R, xm);
    gd = mlp_rows<T>(c, c->wgu[l], c->wd[l], R, xm);
  }
  norm_rows<T>(c, c->x, gd, true, c->ln_f, R, xm, c->tapbuf, rm.seq, c->sd.tap, L);
  g = gemm<T>(c, c->lm_head, c->xn, xm, R, f.vocab, d);
  TOPK_LAUNCH(c, dim3(R, c->tk_nsplit), g, f.vocab, 2, c->tk_nsplit, c->tks, c->top_val, c->top_id, c->lse_rows, logits);
  LAUNCH(c, k_argmax_out, (R + 127) / 128, 128, 0, c->top_id, c->top_val, R, argmax, margin,
         argmax == c->argmax_i ? (int *)nullptr : c->argmax_i);
  return DREAM_OK;
}

extern "C" dream_status dream_verify_tree(dream_ctx *c, const int32_t *seqs, int32_t n_seqs, const dream_tree *trees,
                                          int32_t *node_argmax, float *node_margin, float *logits) {
  TreeBatch tb;
  dream_status s = make_batch(c, seqs, n_seqs, trees, false, &tb);
  if (s) return s;
  if (!node_argmax) return fail(c, DREAM_E_ARG, "node_argmax is required");
  refresh_bounds(c);
  for (int b = 0; b < n_seqs; ++b) {
    if (c->phase[seqs[b]] != PH_DRAFTED) return fail(c, DREAM_E_STATE, "sequence %d: dream_verify_tree follows dream_draft_tree", seqs[b]);
    if (c->p_ub[seqs[b]] + c->T > c->cfg.max_seq) return fail(c, DREAM_E_CAPACITY, "sequence %d may outgrow max_seq", seqs[b]);
  }
  s = c->cfg.dtype == DREAM_BF16 ? verify_impl<bf16>(c, tb, n_seqs, node_argmax, node_margin, logits)
                                 : verify_impl<float>(c, tb, n_seqs, node_argmax, node_margin, logits);
  if (s) return s;
  s = call_done(c);
  if (s) return s;
  for (int b = 0; b < n_seqs; ++b) { c->phase[seqs[b]] = PH_VERIFIED; c->last_verify_seq[b] = seqs[b]; }
  c->last_verify_n = n_seqs;
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- accept

// The tapped features, row map and argmax of a verify are kept by batch slot, so the acceptance must
// name the same sequences in the same order.
static bool same_list_as_verify(const dream_ctx *c, const int *seqs, int n_seqs) {
  if (n_seqs != c->last_verify_n) return false;
  for (int b = 0; b < n_seqs; ++b) if (seqs[b] != c->last_verify_seq[b]) return false;
  return true;
}

template <typename T>
// `logits` null: greedy acceptance on `argmax`; otherwise the sampling form on `logits` at
// temperature `temp` with the caller's `uniforms`.
static dream_status accept_impl(dream_ctx *c, const TreeBatch &tb, int B, const int *argmax, int *accept_len,
                                int *out_tokens, int *comp_src, const float *logits = nullptr, float temp = 0.f,
                                const float *uniforms = nullptr) {
  const dream_config &f = c->cfg;
  int D = c->ts.D, d = f.d_model, R = B * (D + 1);
  RowMeta &rm = c->rm[0];
  if (logits && f.vocab <= 32 * 32 * SAMPLE_CACHE) LAUNCH(c, k_accept_sample<true>, B, 1024, 0, tb, B, c->T, D, f.vocab, c->sd, logits, temp, uniforms, accept_len, out_tokens, comp_src, c->status);
  else if (logits) LAUNCH(c, k_accept_sample<false>, B, 1024, 0, tb, B, c->T, D, f.vocab, c->sd, logits, temp, uniforms, accept_len, out_tokens, comp_src, c->status);
  else LAUNCH(c, k_accept, B, 32, 0, tb, B, c->T, D, c->sd, argmax, accept_len, out_tokens, comp_src);
  LAUNCH(c, (k_compact_kv<T>), dim3(f.n_layers * 2, B), 256, 0, tb, c->sd, c->kv_pool, c->layer_stride, c->kv_stride, paged(c, 0));
  if (c->ent_sum) LAUNCH(c, k_accept_entropy, B, 64, 0, tb, c->T, f.n_layers, f.n_heads, ROW_CHUNK, c->sd, (const float *)c->row_ent, c->ent_sum);
  LAUNCH(c, k_accept_rows, 1, 32, 0, tb, B, c->T, D, c->sd, c->gather_idx, rm, c->cap_rows - c->ts.NI, c->status);
  const XMode xm = xmode(c, R);
  LAUNCH(c, (k_gather_rows<T>), R, 256, 0, c->tapbuf, c->gather_idx, (T *)c->raw, d, (const int *)nullptr, 0, 0LL, xlay(xm, d));
  GemmOut g = gemm<T>(c, c->dw.xkv, c->raw, xm, R, c->kvN, d);
  LAUNCH(c, k_mem_append, dim3(R, (c->kvN + 1023) / 1024), 256, 0, g, rm.seq, rm.dst, (const int *)nullptr, (const int *)nullptr, 0, flat(c, c->dmem));
  return DREAM_OK;
}

extern "C" dream_status dream_accept(dream_ctx *c, const int32_t *seqs, int32_t n_seqs, const dream_tree *trees,
                                     const int32_t *node_argmax, int32_t *accept_len, int32_t *out_tokens,
                                     int32_t *comp_src) {
  TreeBatch tb;
  dream_status s = make_batch(c, seqs, n_seqs, trees, false, &tb);
  if (s) return s;
  if (!node_argmax || !accept_len || !out_tokens) return fail(c, DREAM_E_ARG, "node_argmax, accept_len, out_tokens are required");
  for (int b = 0; b < n_seqs; ++b)
    if (c->phase[seqs[b]] != PH_VERIFIED) return fail(c, DREAM_E_STATE, "sequence %d: dream_accept follows dream_verify_tree", seqs[b]);
  if (!same_list_as_verify(c, seqs, n_seqs)) return fail(c, DREAM_E_STATE, "dream_accept takes the sequence list of the last dream_verify_tree, in the same order");
  s = c->cfg.dtype == DREAM_BF16 ? accept_impl<bf16>(c, tb, n_seqs, node_argmax, accept_len, out_tokens, comp_src)
                                 : accept_impl<float>(c, tb, n_seqs, node_argmax, accept_len, out_tokens, comp_src);
  if (s) return s;
  s = call_done(c);
  if (s) return s;
  for (int b = 0; b < n_seqs; ++b) { c->phase[seqs[b]] = PH_READY; c->p_ub[seqs[b]] += c->ts.D + 1; c->accepts[seqs[b]]++; }
  snapshot_lengths(c);
  return DREAM_OK;
}

extern "C" dream_status dream_accept_sample(dream_ctx *c, const int32_t *seqs, int32_t n_seqs, const dream_tree *trees,
                                            const float *logits, float temperature, const float *uniforms,
                                            int32_t *accept_len, int32_t *out_tokens, int32_t *comp_src) {
  TreeBatch tb;
  dream_status s = make_batch(c, seqs, n_seqs, trees, false, &tb);
  if (s) return s;
  if (!logits || !uniforms || !accept_len || !out_tokens) return fail(c, DREAM_E_ARG, "logits, uniforms, accept_len, out_tokens are required");
  if (!(temperature > 0.f)) return fail(c, DREAM_E_ARG, "temperature must be above zero (dream_accept is the greedy form)");
  for (int b = 0; b < n_seqs; ++b)
    if (c->phase[seqs[b]] != PH_VERIFIED) return fail(c, DREAM_E_STATE, "sequence %d: dream_accept_sample follows dream_verify_tree", seqs[b]);
  if (!same_list_as_verify(c, seqs, n_seqs)) return fail(c, DREAM_E_STATE, "dream_accept_sample takes the sequence list of the last dream_verify_tree, in the same order");
  s = c->cfg.dtype == DREAM_BF16 ? accept_impl<bf16>(c, tb, n_seqs, nullptr, accept_len, out_tokens, comp_src, logits, temperature, uniforms)
                                 : accept_impl<float>(c, tb, n_seqs, nullptr, accept_len, out_tokens, comp_src, logits, temperature, uniforms);
  if (s) return s;
  s = call_done(c);
  if (s) return s;
  for (int b = 0; b < n_seqs; ++b) { c->phase[seqs[b]] = PH_READY; c->p_ub[seqs[b]] += c->ts.D + 1; c->accepts[seqs[b]]++; }
  snapshot_lengths(c);
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- whole step, host results

extern "C" dream_status dream_step_host(dream_ctx *c, const int32_t *seqs, int32_t n_seqs, int32_t *accept_len_host,
                                        int32_t *out_tokens_host) {
  if (!c || !accept_len_host || !out_tokens_host) return fail(c, DREAM_E_ARG, "null argument");
  dream_status s = dream_draft_tree(c, seqs, n_seqs, nullptr);
  if (s) return s;
  s = dream_verify_tree(c, seqs, n_seqs, nullptr, c->argmax_i, c->margin_i, nullptr);
  if (s) return s;
  s = dream_accept(c, seqs, n_seqs, nullptr, c->argmax_i, c->accept_len_i, c->out_tokens_i, c->comp_src_i);
  if (s) return s;
  int D1 = c->ts.D + 1;
  int *stage = c->h_stage + (size_t)c->cfg.max_batch * c->pps;
  CUDA_OK(c, cudaMemcpyAsync(stage, c->accept_len_i, sizeof(int) * n_seqs, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(c, cudaMemcpyAsync(stage + DREAM_MAX_BATCH, c->out_tokens_i, sizeof(int) * n_seqs * D1, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  refresh_bounds(c);                     // the snapshot of this round's accept has landed: the bounds are exact
  memcpy(accept_len_host, stage, sizeof(int) * n_seqs);
  memcpy(out_tokens_host, stage + DREAM_MAX_BATCH, sizeof(int) * n_seqs * D1);
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- read-back

extern "C" dream_status dream_seq_state(dream_ctx *c, int32_t seq, int32_t *verified_len, int32_t *pending, int32_t *tap) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  int P_now = 0;
  CUDA_OK(c, cudaMemcpy(&P_now, c->sd.P + seq, sizeof(int), cudaMemcpyDeviceToHost));
  if (c->phase[seq] >= PH_READY && P_now < c->p_ub[seq]) c->p_ub[seq] = P_now;   // the stream is idle: P is exact
  if (verified_len) *verified_len = P_now;
  if (pending) CUDA_OK(c, cudaMemcpy(pending, c->sd.pending + seq, sizeof(int), cudaMemcpyDeviceToHost));
  if (tap) CUDA_OK(c, cudaMemcpy(tap, c->sd.tap + seq, sizeof(int), cudaMemcpyDeviceToHost));
  return DREAM_OK;
}

extern "C" dream_status dream_layer_entropy(dream_ctx *c, int32_t seq, float *layer_entropy, int32_t *layer_now) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  const dream_config &f = c->cfg;
  if (!c->ent_sum) return fail(c, DREAM_E_STATE, "config.track_entropy is 0");
  if (c->phase[seq] == PH_EMPTY) return fail(c, DREAM_E_STATE, "sequence %d has no prefill", seq);
  std::vector<float> sum(f.n_layers);
  int P = 0;
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  CUDA_OK(c, cudaMemcpy(sum.data(), c->ent_sum + (size_t)seq * f.n_layers, sizeof(float) * f.n_layers, cudaMemcpyDeviceToHost));
  CUDA_OK(c, cudaMemcpy(&P, c->sd.P + seq, sizeof(int), cudaMemcpyDeviceToHost));
  if (P < 1) return fail(c, DREAM_E_STATE, "sequence %d has no verified row", seq);
  const float denom = (float)f.n_heads * (float)P;
  for (int l = 0; l < f.n_layers; ++l) sum[l] /= denom;
  if (layer_entropy) memcpy(layer_entropy, sum.data(), sizeof(float) * f.n_layers);
  if (layer_now) {
    int best = f.tap_layer;
    if (f.tap_mode != DREAM_TAP_FIXED) {
      best = f.tap_lo;                                         // ties go to the lower layer
      for (int l = f.tap_lo + 1; l <= f.tap_hi; ++l) {
        const float a = sum[l - 1], b = sum[best - 1];
        if (f.tap_mode == DREAM_TAP_ENTROPY_MIN ? a < b : a > b) best = l;
      }
    }
    *layer_now = best;
  }
  return DREAM_OK;
}

template <typename T>
static dream_status debug_read_impl(dream_ctx *c, int seq, int what, int layer, int index, float *dst) {
  const dream_config &f = c->cfg;
  int w = f.n_kv_heads * f.head_dim, d = f.d_model;
  float *tmp = c->gout;     // scratch: idle between calls
  int count = what <= 5 || what >= 8 ? w : d;
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  if (what == 0 || what == 1) {
    if (layer < 0 || layer >= f.n_layers || index < 0 || index >= f.max_seq) return fail(c, DREAM_E_ARG, "layer/position out of range");
    if (c->seq_pages[seq].empty()) return fail(c, DREAM_E_STATE, "sequence has no pages");
    int pg = c->seq_pages[seq][index / f.page_tokens], in = index % f.page_tokens;
    const T *base = (const T *)c->kv_pool + (size_t)layer * c->layer_stride + (size_t)what * c->kv_stride;
    const T *src = base + (((size_t)pg * f.n_kv_heads) * f.page_tokens + in) * f.head_dim;
    k_read_row<T><<<f.n_kv_heads, 256, 0, c->stream>>>(src, (long long)f.page_tokens * f.head_dim, tmp, f.head_dim, 0);
  } else if ((what >= 2 && what <= 5) || what == 8 || what == 9) {
    if (index < 0 || index >= c->cap_rows) return fail(c, DREAM_E_ARG, "row out of range");
    if (what >= 8 && !c->three) return fail(c, DREAM_E_STATE, "no final decoder block: draft_blocks is not 3");
    const float *base = what <= 3 ? c->dmem : (what <= 5 ? c->dself : c->dself2);
    int kvsel = (what - 2) & 1;
    // a row holds head_dim floats, or head_dim high then head_dim low bf16 parts: 4 bytes per element either way
    const float *src = base + (((size_t)seq * 2 + kvsel) * f.n_kv_heads * c->cap_rows + index) * f.head_dim;
    const long long hs = (long long)c->cap_rows * f.head_dim;
    if (sizeof(T) == 2) k_read_row<bf16><<<f.n_kv_heads, 256, 0, c->stream>>>((const bf16 *)src, 2 * hs, tmp, f.head_dim, 1);
    else k_read_row<float><<<f.n_kv_heads, 256, 0, c->stream>>>(src, hs, tmp, f.head_dim, 0);
  } else if (what == 6 || what == 7) {
    if (index < 0 || index >= ROW_CHUNK) return fail(c, DREAM_E_ARG, "row out of range");
    const float *src = (what == 6 ? c->tapbuf : c->x) + (size_t)index * d;
    k_read_row<float><<<1, 256, 0, c->stream>>>(src, 0LL, tmp, d, 0);
  } else return fail(c, DREAM_E_ARG, "unknown buffer id %d", what);
  CUDA_OK(c, cudaMemcpyAsync(dst, tmp, sizeof(float) * count, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  return DREAM_OK;
}

// out[r][c] = sum_k X[r][k] W[c][k] through the context's GEMM path (test hook).
__global__ void k_split_rows(const float *src, void *dst, int K, XLayout lay, int is_bf16) {
  kernel_entry(TR_k_split_rows);
  int r = blockIdx.x;
  for (int i = threadIdx.x; i < K; i += blockDim.x) {
    float v = src[(long long)r * K + i];
    if (is_bf16) store_split<bf16>((bf16 *)dst + r * lay.row_stride + i, lay.lo_delta, v);
    else ((float *)dst)[(long long)r * K + i] = v;
  }
}
__global__ void k_gemm_collect(GemmOut g, float *dst, int N) {
  kernel_entry(TR_k_gemm_collect);
  int r = blockIdx.y, c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < N) dst[(long long)r * N + c] = gemm_val(g, r, c);
}

extern "C" dream_status dream_debug_gemm(dream_ctx *c, const void *W, const float *X, int32_t rows, int32_t N,
                                         int32_t K, int32_t split, float *out) {
  if (!c || !W || !X || !out) return fail(c, DREAM_E_ARG, "null argument");
  const dream_config &f = c->cfg;
  bool bf = f.dtype == DREAM_BF16;
  void *buf;
  if (K <= f.d_model) buf = c->xn;
  else if (K <= f.d_ff) buf = c->act;
  else return fail(c, DREAM_E_ARG, "K exceeds the context's widest GEMM input");
  if (rows < 1 || rows > ROW_CHUNK) return fail(c, DREAM_E_ARG, "rows out of range");
  if (bf && (K % 64 || N % 8)) return fail(c, DREAM_E_ARG, "K must be a multiple of 64 and N of 8");
  XMode xm = xmode(c, rows);
  if (bf && !split) {                     // single bf16 row per token
    if (rows > TC_ROWS_MAX) return fail(c, DREAM_E_ARG, "unsplit inputs take at most 128 rows");
    xm = XMode{TC_X_PLAIN, 0};
  }
  size_t need_out = (size_t)rows * N;
  (void)need_out;
  LAUNCH(c, k_split_rows, rows, 256, 0, X, buf, K, xlay(xm, K), bf ? 1 : 0);
  GemmOut g = bf ? gemm<bf16>(c, W, buf, xm, rows, N, K) : gemm<float>(c, W, buf, xm, rows, N, K);
  LAUNCH(c, k_gemm_collect, dim3((N + 255) / 256, rows), 256, 0, g, out, N);
  CUDA_OK(c, cudaGetLastError());
  if (c->gemm_failed) { c->gemm_failed = 0; return fail(c, DREAM_E_UNSUPPORTED, "the GEMM launch was refused (shape or output room)"); }
  return DREAM_OK;
}

// ------------------------------------------------------------------------------------- top-k without an arena

// Scratch of dream_topk_lse_static: partial lists, (m, z) pairs and the per-row block counters of
// k_topk_lse for up to NA_MAX_ROWS rows and NA_MAX_SPLIT vocabulary blocks.  It lives in the
// library image, so every GPU that loads the library holds these ~1.1 MB until the process exits.
#define NA_MAX_ROWS 128
#define NA_MAX_SPLIT 64
struct NaScratch {
  float pv[NA_MAX_ROWS * NA_MAX_SPLIT * TOPK_MAX];
  int pi[NA_MAX_ROWS * NA_MAX_SPLIT * TOPK_MAX];
  float pm[NA_MAX_ROWS * NA_MAX_SPLIT];
  float pz[NA_MAX_ROWS * NA_MAX_SPLIT];
  int counter[NA_MAX_ROWS];
};
static __device__ __align__(256) unsigned char g_na_scratch[sizeof(NaScratch)];
// In host code g_na_scratch is only a handle; the address a kernel can use comes from
// cudaGetSymbolAddress, looked up once per device.
#define NA_MAX_DEVICES 64
static NaScratch *g_na_dev_ptr[NA_MAX_DEVICES];

extern "C" dream_status dream_topk_lse_static(const float *logits, int32_t rows, int32_t vocab, int32_t ktop,
                                              float *top_val, int32_t *top_id, float *lse, void *cuda_stream) {
  if (!logits || !top_val || !top_id || !lse) return fail(nullptr, DREAM_E_ARG, "dream_topk_lse_static: null buffer");
  if (rows < 1 || rows > NA_MAX_ROWS)
    return fail(nullptr, DREAM_E_CAPACITY, "dream_topk_lse_static: rows = %d outside 1..%d (the built-in scratch is fixed)", rows, NA_MAX_ROWS);
  if (vocab < 2 || vocab > NA_MAX_SPLIT * TOPK_COLS)
    return fail(nullptr, DREAM_E_CAPACITY, "dream_topk_lse_static: vocab = %d outside 2..%d (the built-in scratch is fixed)", vocab, NA_MAX_SPLIT * TOPK_COLS);
  if (ktop < 1 || ktop > TOPK_MAX || ktop > vocab)
    return fail(nullptr, DREAM_E_ARG, "dream_topk_lse_static: ktop = %d outside 1..%d", ktop, TOPK_MAX);
  if ((uintptr_t)logits & 15) return fail(nullptr, DREAM_E_ARG, "dream_topk_lse_static: logits must be 16-byte aligned");
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(nullptr, DREAM_E_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= NA_MAX_DEVICES) return fail(nullptr, DREAM_E_UNSUPPORTED, "device ordinal %d not supported", dev);
  if (!g_na_dev_ptr[dev]) {                    // first call on this device, with it current
    void *ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_na_scratch);
    if (e != cudaSuccess || !ptr) return fail(nullptr, DREAM_E_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    g_na_dev_ptr[dev] = (NaScratch *)ptr;
  }
  NaScratch *sc = g_na_dev_ptr[dev];
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // the scratch keeps whatever the last call left: only the block counters have to start at zero
  e = cudaMemsetAsync(sc->counter, 0, sizeof(int) * rows, stream);
  if (e != cudaSuccess) return fail(nullptr, DREAM_E_CUDA, "clearing the counters: %s", cudaGetErrorString(e));
  TopkScratch ts;
  ts.pv = sc->pv; ts.pi = sc->pi; ts.pm = sc->pm; ts.pz = sc->pz; ts.counter = sc->counter;
  GemmOut g;                                   // a plain [rows][vocab] matrix: one slot, one chunk
  g.base = logits; g.slot_stride = 0; g.chunk_stride = 0; g.chunk_shift = 30; g.ld = vocab; g.kb = 0; g.upc = 0;
  int nsplit = (vocab + TOPK_COLS - 1) / TOPK_COLS;
  k_topk_lse<TOPK_COLS / TOPK_THREADS><<<dim3(rows, nsplit), TOPK_THREADS, 0, stream>>>(g, vocab, ktop, nsplit, ts, top_val, top_id, lse, (float *)nullptr);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, DREAM_E_CUDA, "k_topk_lse launch: %s", cudaGetErrorString(e));
  return DREAM_OK;
}

static const char *const g_trace_names[] = DREAM_TRACE_NAMES;

extern "C" dream_status dream_trace(dream_ctx *c, unsigned long long *buffer, int64_t capacity_entries) {
  if (!c) return DREAM_E_ARG;
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  unsigned long long *ptr = nullptr;
  if (buffer) {
    if (capacity_entries < 1) return fail(c, DREAM_E_ARG, "trace capacity");
    unsigned long long head[2] = {0ull, (unsigned long long)capacity_entries};
    CUDA_OK(c, cudaMemcpy(buffer, head, sizeof(head), cudaMemcpyHostToDevice));
    ptr = buffer;
  }
  CUDA_OK(c, cudaMemcpyToSymbol(g_dream_trace, &ptr, sizeof(ptr)));
  return DREAM_OK;
}

extern "C" const char *dream_trace_name(int32_t id) {
  return id >= 0 && id < TR_count ? g_trace_names[id] : "?";
}

extern "C" dream_status dream_gemm_timing(dream_ctx *c, int32_t on, int64_t *launches, double *total_ms, double *weight_bytes) {
  if (!c) return DREAM_E_ARG;
  if (on) {
    const int cap = 8192;                       // timed launches per measurement window
    while ((int)c->prof_ev.size() < 2 * cap) {
      cudaEvent_t e;
      CUDA_OK(c, cudaEventCreate(&e));
      c->prof_ev.push_back(e);
    }
    c->prof_on = 1; c->prof_n = 0; c->prof_bytes = 0.0;
    return DREAM_OK;
  }
  c->prof_on = 0;
  CUDA_OK(c, cudaStreamSynchronize(c->stream));
  double ms = 0.0;
  for (int i = 0; i < c->prof_n; ++i) {
    float t = 0.f;
    CUDA_OK(c, cudaEventElapsedTime(&t, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]));
    ms += t;
  }
  if (launches) *launches = c->prof_n;
  if (total_ms) *total_ms = ms;
  if (weight_bytes) *weight_bytes = c->prof_bytes;
  return DREAM_OK;
}

extern "C" dream_status dream_gemm_counts(const dream_ctx *c, int64_t *tensor_core, int64_t *cuda_core) {
  if (!c) return DREAM_E_ARG;
  if (tensor_core) *tensor_core = c->tc_launches;
  if (cuda_core) *cuda_core = c->simt_launches;
  return DREAM_OK;
}

extern "C" dream_status dream_debug_read(dream_ctx *c, int32_t seq, int32_t what, int32_t layer, int32_t index, float *dst) {
  dream_status s = check_seq(c, seq);
  if (s) return s;
  if (!dst) return fail(c, DREAM_E_ARG, "null destination");
  return c->cfg.dtype == DREAM_BF16 ? debug_read_impl<bf16>(c, seq, what, layer, index, dst)
                                    : debug_read_impl<float>(c, seq, what, layer, index, dst);
}
