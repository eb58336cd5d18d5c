// Integer side of the loop: per-sequence state, tree expansion and re-ranking
// (Section 3.1, tree drafting; Section 4: depth, children per node, maximum draft length),
// verification row set-up, greedy acceptance (Section 2.1) and KV-cache compaction.
#pragma once
#include "common.cuh"
#include "rows.cuh"

#define DREAM_MAX_DEPTH 15

// Per-sequence device state (arrays indexed by sequence id).
struct SeqDev {
  int *P;            // verified length: target KV slots [0, P) are final
  int *pending;      // token at position P (known, not yet run through the target)
  int *tap;          // selected feature layer l* (1-based)
  int *nperm_d;      // permanent rows of the draft self-attention cache
  int *nperm_m;      // permanent rows of the cross-attention memory
  int *n_new;        // tokens verified by the last accept, still without draft K/V rows
  int *new_tok;      // [seq][DREAM_MAX_DEPTH+1]
  int *new_pos;      // [seq][DREAM_MAX_DEPTH+1]
  int *last_P;       // P before the last accept
  int *last_A;       // accepted draft tokens of the last accept
  int *path;         // [seq][DREAM_MAX_DEPTH+1] tree nodes on the accepted path
};

// Static shape of the draft tree for one configuration (host-computed).
struct TreeShape {
  int D, K, N, T;                       // depth, children per node, node cap, nodes incl. root
  int beam[DREAM_MAX_DEPTH + 1];        // beam[p] = nodes expanded in pass p+1 (beam[0] = 1)
  int in_off[DREAM_MAX_DEPTH + 1];      // first input-node index of pass p+1
  int cand_off[DREAM_MAX_DEPTH + 1];    // first candidate index created by pass p+1
  int NI, NC;                           // input nodes and candidates in total
};

// Draft-side tree storage of all sequences (device).
struct DraftTreeDev {
  int *in_tok, *in_depth, *in_cand;     // [seq][NI]
  float *in_cum;                        // [seq][NI]
  unsigned long long *in_anc;           // [seq][NI] ancestor-or-self bits over input nodes
  int *cand_tok, *cand_par, *cand_depth;  // [seq][NC]; cand_par = candidate index or -1 (root)
  float *cand_cum;                      // [seq][NC]
};

// Row metadata of the current launch set.
struct RowMeta {
  int *seq, *tok, *pos, *slot, *dst, *in;
  // Three-block draft: a row with vis_d >= 0 is a permanent row (context or catch-up): it sees the
  // first vis_d rows of the self-attention caches and the first vis_m memory rows, nothing else.
  int *vis_d, *vis_m;
};

struct TreePtrs {                       // device buffers of one caller-visible tree
  int *tokens, *parent, *depth;
  uint32_t *mask;
  float *cum;
};
struct TreeBatch { TreePtrs t[DREAM_MAX_BATCH]; int seq[DREAM_MAX_BATCH]; };

// ---------------------------------------------------------------------------------------
// Start of a draft call: row set of pass 1 = [root, catch-up rows...] per sequence.
// The catch-up rows are the tokens verified by the last accept; they receive permanent
// draft self-attention K/V rows.  One thread per sequence slot b.
__global__ void k_draft_begin(TreeBatch tb, int B, SeqDev s, DraftTreeDev dt, TreeShape ts,
                              RowMeta rm, int rows_per_seq, int cap_rows, int *status) {
  // Visibility of the catch-up rows (read by the three-block draft only): catch-up row j sits at
  // position P_old + j, behind np + j rows of the self-attention caches; the acceptance appended one
  // memory row per catch-up token, so the memory rows of earlier positions are the first nm - nn + j.
  kernel_entry(TR_k_draft_begin);
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int seq = tb.seq[b];
  int P = s.P[seq], nn = s.n_new[seq], np = s.nperm_d[seq];
  if (np + nn + ts.NI > cap_rows || s.nperm_m[seq] + ts.NI > cap_rows) {
    atomicMax(status, DREAM_DEV_BAD_INDEX);
    nn = 0;
  }
  int base = b * rows_per_seq;
  for (int j = 0; j < rows_per_seq; ++j) {
    int r = base + j;
    rm.seq[r] = seq;
    rm.vis_d[r] = -1; rm.vis_m[r] = -1;
    if (j == 0) {
      rm.tok[r] = s.pending[seq]; rm.pos[r] = P; rm.dst[r] = np + nn; rm.in[r] = 0;
    } else if (j - 1 < nn) {
      rm.tok[r] = s.new_tok[seq * (DREAM_MAX_DEPTH + 1) + j - 1];
      rm.pos[r] = s.new_pos[seq * (DREAM_MAX_DEPTH + 1) + j - 1];
      rm.dst[r] = np + j - 1; rm.in[r] = -1;
      rm.vis_d[r] = np + j; rm.vis_m[r] = max(0, s.nperm_m[seq] - nn + j - 1);
    } else {
      rm.tok[r] = -1; rm.pos[r] = 0; rm.dst[r] = -1; rm.in[r] = -1;
    }
  }
  s.nperm_d[seq] = np + nn;
  s.n_new[seq] = 0;
  long long o = (long long)seq * ts.NI;
  dt.in_tok[o] = s.pending[seq]; dt.in_depth[o] = 0; dt.in_cand[o] = -1;
  dt.in_cum[o] = 0.f; dt.in_anc[o] = 1ull;
}

// After pass `p` (1-based): turn the per-row top-K into candidates, pick the next beam.
// One block per sequence slot.  Rows of this pass: row b*rows_per_seq + i expands input
// node in_off[p-1] + i, i < beam[p-1].
__global__ void k_tree_expand(TreeBatch tb, SeqDev s, DraftTreeDev dt, TreeShape ts, int p,
                              int rows_per_seq, const float *__restrict__ top_val,
                              const int *__restrict__ top_id, const float *__restrict__ lse,
                              RowMeta rm_next, int next_rows_per_seq) {
  kernel_entry(TR_k_tree_expand);
  __shared__ float cum[256];
  int b = blockIdx.x, seq = tb.seq[b];
  int K = ts.K, m = ts.beam[p - 1], nnew = m * K;
  long long io = (long long)seq * ts.NI, co = (long long)seq * ts.NC;
  int c0 = ts.cand_off[p - 1];
  for (int t = threadIdx.x; t < nnew; t += blockDim.x) {
    int i = t / K, j = t - i * K;
    int node = ts.in_off[p - 1] + i, r = b * rows_per_seq + i;
    float cm = dt.in_cum[io + node] + (top_val[r * K + j] - lse[r]);
    dt.cand_tok[co + c0 + t] = top_id[r * K + j];
    dt.cand_par[co + c0 + t] = dt.in_cand[io + node];
    dt.cand_depth[co + c0 + t] = dt.in_depth[io + node] + 1;
    dt.cand_cum[co + c0 + t] = cm;
    cum[t] = cm;
  }
  __syncthreads();
  if (p >= ts.D) return;
  int nb = ts.beam[p], P = s.P[seq], np = s.nperm_d[seq];
  for (int t = threadIdx.x; t < nnew; t += blockDim.x) {
    int rank = 0;
    for (int u = 0; u < nnew; ++u) rank += better(cum[u], u, cum[t], t) ? 1 : 0;
    if (rank >= nb) continue;
    int i = t / K, par_in = ts.in_off[p - 1] + i, me = ts.in_off[p] + rank;
    dt.in_tok[io + me] = dt.cand_tok[co + c0 + t];
    dt.in_depth[io + me] = p;
    dt.in_cand[io + me] = c0 + t;
    dt.in_cum[io + me] = cum[t];
    dt.in_anc[io + me] = dt.in_anc[io + par_in] | (1ull << me);
    int r = b * next_rows_per_seq + rank;
    rm_next.seq[r] = seq; rm_next.tok[r] = dt.cand_tok[co + c0 + t]; rm_next.pos[r] = P + p;
    rm_next.dst[r] = np + me; rm_next.in[r] = me;
  }
  for (int t = nb + threadIdx.x; t < next_rows_per_seq; t += blockDim.x) {   // idle tail rows
    int r = b * next_rows_per_seq + t;
    rm_next.seq[r] = seq; rm_next.tok[r] = -1; rm_next.pos[r] = 0; rm_next.dst[r] = -1; rm_next.in[r] = -1;
  }
}

// After the last pass: keep the N best candidates by cumulative log-probability (ties ->
// earlier candidate), order them by creation index behind the root, remap parents, build
// the ancestor-or-self masks.  One block per sequence slot.
__global__ void k_tree_finalize(TreeBatch tb, SeqDev s, DraftTreeDev dt, TreeShape ts) {
  kernel_entry(TR_k_tree_finalize);
  extern __shared__ int sm[];
  int NC = ts.NC, Nsel = ts.T - 1;
  int *sel = sm, *node_of = sm + NC;       // [NC] each
  int b = blockIdx.x, seq = tb.seq[b];
  long long co = (long long)seq * ts.NC;
  TreePtrs tp = tb.t[b];
  for (int t = threadIdx.x; t < NC; t += blockDim.x) {
    float ct = dt.cand_cum[co + t];
    int rank = 0;
    for (int u = 0; u < NC; ++u) rank += better(dt.cand_cum[co + u], u, ct, t) ? 1 : 0;
    sel[t] = rank < Nsel ? 1 : 0;
  }
  __syncthreads();
  for (int t = threadIdx.x; t < NC; t += blockDim.x) {
    int before = 0;
    for (int u = 0; u < t; ++u) before += sel[u];
    node_of[t] = sel[t] ? before + 1 : -1;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    tp.tokens[0] = s.pending[seq]; tp.parent[0] = -1; tp.depth[0] = 0;
    if (tp.cum) tp.cum[0] = 0.f;
    tp.mask[0] = 1u; tp.mask[1] = 0u; tp.mask[2] = 0u; tp.mask[3] = 0u;
  }
  for (int t = threadIdx.x; t < NC; t += blockDim.x) {
    int me = node_of[t];
    if (me < 0) continue;
    int par = dt.cand_par[co + t];
    tp.tokens[me] = dt.cand_tok[co + t];
    tp.parent[me] = par < 0 ? 0 : node_of[par];
    tp.depth[me] = dt.cand_depth[co + t];
    if (tp.cum) tp.cum[me] = dt.cand_cum[co + t];
    uint32_t mk[4] = {1u, 0u, 0u, 0u};               // the root is everyone's ancestor
    int a = t;
    while (a >= 0) { int na = node_of[a]; mk[na >> 5] |= 1u << (na & 31); a = dt.cand_par[co + a]; }
    for (int wd = 0; wd < 4; ++wd) tp.mask[me * 4 + wd] = mk[wd];
  }
}


// What an acceptance leaves behind for sequence slot b: the emitted tokens (A accepted draft
// tokens, then the target's own token g), the compaction map, the tokens that still lack draft
// K/V rows, and the advanced prefix.  One thread.
__device__ __forceinline__ void accept_commit(const TreePtrs &tp, int b, int seq, int D, const SeqDev &s, const int *path,
                                              int A, int g, int *accept_len, int *out_tokens, int *comp_src) {
  int P = s.P[seq];
  out_tokens[b * (D + 1) + A] = g;
  for (int j = A + 1; j <= D; ++j) out_tokens[b * (D + 1) + j] = -1;
  accept_len[b] = A;
  for (int j = 0; j <= D; ++j) {
    if (comp_src) comp_src[b * (D + 1) + j] = j <= A ? path[j] : -1;
    if (j <= A) {
      s.new_tok[seq * (DREAM_MAX_DEPTH + 1) + j] = tp.tokens[path[j]];
      s.new_pos[seq * (DREAM_MAX_DEPTH + 1) + j] = P + j;
    }
  }
  s.n_new[seq] = A + 1;
  s.last_P[seq] = P; s.last_A[seq] = A;
  s.P[seq] = P + A + 1;
  s.pending[seq] = g;
}

// ---------------------------------------------------------------------------------------
// Verification rows: node i of slot b is row b*T + i at position P + depth[i], KV slot P + i.
__global__ void k_verify_setup(TreeBatch tb, int B, int T, SeqDev s, RowMeta rm, uint32_t *mask,
                               int max_seq, int *status) {
  kernel_entry(TR_k_verify_setup);
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= B * T) return;
  int b = r / T, i = r - b * T, seq = tb.seq[b];
  TreePtrs tp = tb.t[b];
  int P = s.P[seq], dep = tp.depth[i], par = tp.parent[i];
  bool bad = (i == 0 ? par != -1 || dep != 0 : par < 0 || par >= i || dep != tp.depth[par < 0 ? 0 : par] + 1);
  if (P + T > max_seq) bad = true;
  if (bad) atomicMax(status, DREAM_DEV_BAD_INDEX);
  // a malformed node keeps its row (so the launch shapes hold) but writes no K/V: slot -1
  rm.seq[r] = seq; rm.tok[r] = tp.tokens[i]; rm.pos[r] = P + (bad ? 0 : dep);
  rm.slot[r] = bad ? -1 : P + i; rm.in[r] = i;
  for (int wd = 0; wd < 4; ++wd) mask[r * 4 + wd] = tp.mask[i * 4 + wd];
}

// Greedy acceptance (Section 2.1): from the root, move to the child whose token equals the
// current node's target argmax; stop when there is none.  Emits the accepted tokens plus
// the target's own token, records the path, and advances the sequence state.
// One warp per sequence slot.
__global__ void k_accept(TreeBatch tb, int B, int T, int D, SeqDev s, const int *__restrict__ argmax,
                         int *accept_len, int *out_tokens, int *comp_src) {
  kernel_entry(TR_k_accept);
  int b = blockIdx.x, lane = threadIdx.x, seq = tb.seq[b];
  TreePtrs tp = tb.t[b];
  const int *am = argmax + b * T;
  int cur = 0, A = 0;
  int *path = s.path + seq * (DREAM_MAX_DEPTH + 1);
  if (lane == 0) path[0] = 0;
  while (A < D) {
    int g = am[cur], found = 0x7fffffff;
    for (int i = 1 + lane; i < T; i += 32)
      if (tp.parent[i] == cur && tp.tokens[i] == g) found = min(found, i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
    if (found == 0x7fffffff) break;
    cur = found; ++A;
    if (lane == 0) { path[A] = cur; out_tokens[b * (D + 1) + A - 1] = tp.tokens[cur]; }
  }
  if (lane == 0) accept_commit(tp, b, seq, D, s, path, A, am[cur], accept_len, out_tokens, comp_src);
}

// ---------------------------------------------------------------------------------------
// Acceptance at a temperature above zero (Section 2.1: a draft token is kept with probability
// min(1, P_target / P_draft); Section 4 evaluates Temp = 1).  The tree's children are the draft's
// top-K choices, i.e. point-mass proposals (P_draft = 1): child c of the current node is kept
// when u < p(token_c), p = softmax(logits[cur] / temp) without the tokens already refused at this
// node, renormalised; children are tried in node order.  When every child is refused (or there is
// none) the emitted token is drawn from what is left of p by inverting its cumulative sum in
// token order.  uniforms[b][j][r]: the number used at path step j for the r-th child tried
// (r < T - 1), [j][T - 1] for the final draw.  One block of 1024 threads per sequence slot; warp
// w owns the tokens [w * seg, (w + 1) * seg).
// CACHED (vocab <= 32768): a thread keeps the exponentials of its up to 32 tokens of the current row
// in registers, so a trial costs no pass over memory; a refused token is zeroed in place.
#define SAMPLE_MAX_REFUSED 128
#define SAMPLE_CACHE 32
template <bool CACHED>
__global__ void __launch_bounds__(1024)
k_accept_sample(TreeBatch tb, int B, int T, int D, int V, SeqDev s, const float *__restrict__ logits, float temp,
                const float *__restrict__ uniforms, int *accept_len, int *out_tokens, int *comp_src, int *status) {
  kernel_entry(TR_k_accept);
  __shared__ float sh[33];
  __shared__ float wtot[32];
  __shared__ int refused[SAMPLE_MAX_REFUSED];
  __shared__ int sh_i[4];
  __shared__ float sh_f[2];
  const int b = blockIdx.x, seq = tb.seq[b], lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const TreePtrs tp = tb.t[b];
  const float inv_t = 1.f / temp;
  const int seg = (((V + 31) / 32) + 31) & ~31;
  const int v0 = w * seg, v1 = min(V, v0 + seg);
  int *path = s.path + seq * (DREAM_MAX_DEPTH + 1);
  if (threadIdx.x == 0) path[0] = 0;
  int cur = 0, A = 0, emitted = -1;
  float ev[CACHED ? SAMPLE_CACHE : 1];
  // at most D + 1 nodes are visited: every pass either walks into a child (A grows, and at A == D
  // no child is looked for) or ends with the final draw, which always emits a token
  for (int visit = 0; visit <= D && emitted < 0; ++visit) {
    const float *row = logits + ((long long)b * T + cur) * V;
    const float *u = uniforms + ((long long)b * (D + 1) + A) * T;
    // the row's maximum (of the scaled logits)
    float m = -INFINITY;
    if (CACHED) {
#pragma unroll
      for (int k = 0; k < SAMPLE_CACHE; ++k) {
        int v = v0 + 32 * k + lane;
        ev[k] = v < v1 ? row[v] * inv_t : -INFINITY;
        m = fmaxf(m, ev[k]);
      }
    } else {
      for (int v = threadIdx.x; v < V; v += blockDim.x) m = fmaxf(m, row[v] * inv_t);
    }
    m = warp_max(m);
    __syncthreads();
    if (lane == 0) sh[w] = m;
    __syncthreads();
    m = sh[0];
    for (int i = 1; i < 32; ++i) m = fmaxf(m, sh[i]);
    if (CACHED) {
#pragma unroll
      for (int k = 0; k < SAMPLE_CACHE; ++k) ev[k] = v0 + 32 * k + lane < v1 ? __expf(ev[k] - m) : 0.f;
    }
    int n_ref = 0, last_kid = 0, tried = 0, taken = -1;
    for (;;) {
      // mass of every token not refused so far, per warp segment, then the whole row
      float acc = 0.f;
      if (CACHED) {
#pragma unroll
        for (int k = 0; k < SAMPLE_CACHE; ++k) acc += ev[k];
      } else {
        for (int v = v0 + lane; v < v1; v += 32) {
          float e = __expf(row[v] * inv_t - m);
          for (int i = 0; i < n_ref; ++i) if (refused[i] == v) e = 0.f;
          acc += e;
        }
      }
      acc = warp_sum(acc);
      __syncthreads();
      if (lane == 0) wtot[w] = acc;
      // next child of cur in node order
      int kid = 0x7fffffff;
      if (A < D)
        for (int i = last_kid + 1 + (int)threadIdx.x; i < T; i += blockDim.x)
          if (tp.parent[i] == cur) kid = min(kid, i);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) kid = min(kid, __shfl_xor_sync(0xffffffffu, kid, o));
      if (lane == 0) sh[w] = __int_as_float(kid);
      __syncthreads();
      if (threadIdx.x == 0) {
        float Z = 0.f;
        for (int i = 0; i < 32; ++i) Z += wtot[i];
        int k = 0x7fffffff;
        for (int i = 0; i < 32; ++i) k = min(k, __float_as_int(sh[i]));
        int decision = 0;                                   // 0 = final draw, 1 = kept, 2 = refused, 3 = no mass
        if (!(Z > 0.f) || Z > 3.0e38f) decision = 3;         // a row of NaN or infinities, or every massive token refused
        else if (k != 0x7fffffff && n_ref < SAMPLE_MAX_REFUSED) {
          int tok = tp.tokens[k];
          float e = (tok >= 0 && tok < V) ? __expf(row[tok] * inv_t - m) : 0.f;
          for (int i = 0; i < n_ref; ++i) if (refused[i] == tok) e = 0.f;
          decision = u[tried] * Z < e ? 1 : 2;
          if (decision == 2) refused[n_ref] = tok;
        }
        sh_i[0] = decision; sh_i[1] = k; sh_f[0] = Z;
      }
      __syncthreads();
      const int decision = sh_i[0];
      if (decision == 0 || decision == 3) break;
      last_kid = sh_i[1];
      ++tried;
      if (decision == 1) { taken = last_kid; break; }
      if (CACHED) {                                         // the owner of the refused token drops it
        const int off = refused[n_ref] - v0;
        if (off >= 0 && off < seg && (off & 31) == lane) {
#pragma unroll
          for (int k = 0; k < SAMPLE_CACHE; ++k) if (k == (off >> 5)) ev[k] = 0.f;
        }
      }
      ++n_ref;
    }
    if (taken >= 0) {
      cur = taken; ++A;
      if (threadIdx.x == 0) { path[A] = cur; out_tokens[b * (D + 1) + A - 1] = tp.tokens[cur]; }
      continue;
    }
    if (sh_i[0] == 3) {                                     // nothing to draw from: token 0, and the status word says so
      if (threadIdx.x == 0) atomicMax(status, DREAM_DEV_BAD_INDEX);
      emitted = 0;
      break;
    }
    // final draw: the first token, in token order, at which the running mass exceeds u * Z
    const float target = u[T - 1] * sh_f[0];
    if (threadIdx.x == 0) {
      float c = 0.f;
      int ws = -1;
      for (int i = 0; i < 32; ++i) { if (c + wtot[i] > target) { ws = i; break; } c += wtot[i]; }
      if (ws < 0) {                                         // rounding pushed the target past the end:
        ws = 31;                                            // the last token that has mass
        while (ws > 0 && wtot[ws] <= 0.f) --ws;
        c = -INFINITY;
      }
      sh_i[2] = ws; sh_f[1] = c;
    }
    __syncthreads();
    if (w == sh_i[2]) {
      float c = sh_f[1];
      int found = -1, last_pos = -1;
      auto group = [&](int base, float e) {
        float inc = e;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { float t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        unsigned hit = __ballot_sync(0xffffffffu, e > 0.f && c + inc > target);
        unsigned pos = __ballot_sync(0xffffffffu, e > 0.f);
        if (pos) last_pos = base + 31 - __clz(pos);
        if (hit && found < 0) found = base + __ffs(hit) - 1;
        c += __shfl_sync(0xffffffffu, inc, 31);
      };
      if (CACHED) {
#pragma unroll
        for (int k = 0; k < SAMPLE_CACHE; ++k)
          if (found < 0 && v0 + 32 * k < v1) group(v0 + 32 * k, ev[k]);
      } else {
        for (int base = v0; base < v1 && found < 0; base += 32) {
          int v = base + lane;
          float e = 0.f;
          if (v < v1) {
            e = __expf(row[v] * inv_t - m);
            for (int i = 0; i < n_ref; ++i) if (refused[i] == v) e = 0.f;
          }
          group(base, e);
        }
      }
      if (found < 0) found = last_pos;                      // the segment's last token with mass
      if (lane == 0) sh_i[3] = found;
    }
    __syncthreads();
    emitted = sh_i[3];
    if (emitted < 0) {                                      // no token with mass was met (cannot happen with Z > 0)
      if (threadIdx.x == 0) atomicMax(status, DREAM_DEV_BAD_INDEX);
      emitted = 0;
    }
  }
  if (emitted < 0) emitted = 0;
  if (threadIdx.x == 0) accept_commit(tp, b, seq, D, s, path, A, emitted, accept_len, out_tokens, comp_src);
}

// KV compaction: the rows of path node j move from tail slot P + path[j] to P + j, for every
// layer and both K and V.  path[j] >= j and strictly increasing, and each thread owns one
// element offset across all rows, so the ascending in-place copy is race-free.
// grid (L*2, B); also fills the row map for the memory-append GEMM that follows.
template <typename T>
__global__ void k_compact_kv(TreeBatch tb, SeqDev s, void *pool, long long layer_stride,
                             long long kv_stride, PagedKV kv) {
  kernel_entry(TR_k_compact_kv);
  int b = blockIdx.y, seq = tb.seq[b];
  int layer = blockIdx.x >> 1, which = blockIdx.x & 1;
  T *base = (T *)pool + (long long)layer * layer_stride + (long long)which * kv_stride;
  int P = s.last_P[seq], A = s.last_A[seq];
  const int *path = s.path + seq * (DREAM_MAX_DEPTH + 1);
  int w = kv.hkv * kv.hd;
  for (int e = threadIdx.x; e < w; e += blockDim.x) {
    int h = e / kv.hd, x = e - h * kv.hd;
    for (int j = 1; j <= A; ++j) {
      int src = path[j];
      if (src == j) continue;
      base[kv.off(seq, P + j, h) + x] = base[kv.off(seq, P + src, h) + x];
    }
  }
}

// Row map for the cross-memory append after an accept: row b*(D+1)+j takes the tapped
// features of path node j (tap-buffer row b*T + path[j]) and lands in memory row
// nperm_m + j.  Then nperm_m advances.  One thread per sequence slot.
__global__ void k_accept_rows(TreeBatch tb, int B, int T, int D, SeqDev s, int *gather_idx,
                              RowMeta rm, int cap_rows, int *status) {
  kernel_entry(TR_k_accept_rows);
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int seq = tb.seq[b], A = s.last_A[seq], nm = s.nperm_m[seq];
  if (nm + A + 1 > cap_rows) { atomicMax(status, DREAM_DEV_BAD_INDEX); A = -1; }
  for (int j = 0; j <= D; ++j) {
    int r = b * (D + 1) + j;
    rm.seq[r] = seq;
    gather_idx[r] = j <= A ? b * T + s.path[seq * (DREAM_MAX_DEPTH + 1) + j] : -1;
    rm.dst[r] = j <= A ? nm + j : -1;
  }
  s.nperm_m[seq] = nm + A + 1;
}

// ---------------------------------------------------------------------------------------
// Tap-layer selection (Section 3.2): argmin (or argmax) of AE over [lo, hi], ties -> lower layer.
__global__ void k_select_tap(const float *__restrict__ ae, int mode, int fixed, int lo, int hi,
                             int *tap_out, int *tap_user) {
  kernel_entry(TR_k_select_tap);
  if (threadIdx.x || blockIdx.x) return;
  int best = fixed;
  if (mode != 0) {
    best = lo;
    for (int l = lo + 1; l <= hi; ++l) {
      float a = ae[l - 1], bb = ae[best - 1];
      if (mode == 1 ? a < bb : a > bb) best = l;
    }
  }
  *tap_out = best;
  if (tap_user) *tap_user = best;
}

// Visual-token selection (Section 3.3): the k visual tokens with the largest importance (ties
// -> lower index), returned ascending; then the compressed context C = kept visual
// positions plus all text positions, ascending.  One block.
__global__ void k_select_visual(const float *__restrict__ scores_all, long long layer_stride,
                                const int *__restrict__ tap, int tap_lo, int v, int k, int vis_start,
                                int n, const int *__restrict__ forced, int *kept, float *scores_out,
                                int *ctx_pos, int *flags /* [n] scratch */) {
  kernel_entry(TR_k_select_visual);
  const float *sc = scores_all + (long long)(*tap - tap_lo) * layer_stride;
  for (int j = threadIdx.x; j < n; j += blockDim.x) flags[j] = (j < vis_start || j >= vis_start + v) ? 1 : 0;
  __syncthreads();
  if (forced) {
    for (int j = threadIdx.x; j < k; j += blockDim.x) flags[vis_start + forced[j]] = 1;
  } else {
    for (int j = threadIdx.x; j < v; j += blockDim.x) {
      float sj = sc[j];
      int rank = 0;
      for (int u = 0; u < v; ++u) rank += better(sc[u], u, sj, j) ? 1 : 0;
      if (rank < k) flags[vis_start + j] = 1;
    }
  }
  for (int j = threadIdx.x; j < v; j += blockDim.x) if (scores_out) scores_out[j] = sc[j];
  __syncthreads();
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    if (!flags[j]) continue;
    int before = 0;
    for (int u = 0; u < j; ++u) before += flags[u];
    ctx_pos[before] = j;
    if (j >= vis_start && j < vis_start + v && kept) {
      int bv = 0;
      for (int u = vis_start; u < j; ++u) bv += flags[u];
      kept[bv] = j - vis_start;
    }
  }
}

// Eq. 2 over the longer sequence (Section 3.2, "during each decoding step"): the entropies of the
// rows an acceptance commits (tree nodes path[0..A] of the sequence in batch slot b) are added to
// the per-layer sums, heads in ascending order inside a row, rows in path order.
// row_ent [L][rows_cap][H] from the last verification; ent_sum [seq][L].  grid (slots), a thread per layer.
__global__ void k_accept_entropy(TreeBatch tb, int T, int L, int H, int rows_cap, SeqDev s,
                                 const float *__restrict__ row_ent, float *ent_sum) {
  kernel_entry(TR_k_accept);
  const int b = blockIdx.x, seq = tb.seq[b], A = s.last_A[seq];
  const int *path = s.path + seq * (DREAM_MAX_DEPTH + 1);
  for (int l = threadIdx.x; l < L; l += blockDim.x) {
    float sum = 0.f;
    for (int j = 0; j <= A; ++j) {
      const float *e = row_ent + ((long long)l * rows_cap + b * T + path[j]) * H;
      for (int h = 0; h < H; ++h) sum += e[h];
    }
    ent_sum[(long long)seq * L + l] += sum;
  }
}

// Row maps of the context-building GEMMs after compression: row i <-> context position
// ctx_pos[i] (or position i when the memory keeps every prompt position).
// mem_all_positions: the memory keeps every prompt position, so a context row at position p has p
// memory rows of earlier positions; otherwise the memory rows are the context rows themselves.
__global__ void k_ctx_rows(const int *__restrict__ ctx_pos, int count, int identity, int seq,
                           RowMeta rm, int *gather_idx, int row0, int mem_all_positions) {
  kernel_entry(TR_k_ctx_rows);
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  int p = identity ? row0 + i : ctx_pos[i];
  rm.seq[i] = seq; rm.pos[i] = p; rm.dst[i] = row0 + i; gather_idx[i] = p;
  rm.in[i] = -1; rm.vis_d[i] = row0 + i + 1; rm.vis_m[i] = mem_all_positions ? p : row0 + i;
}
