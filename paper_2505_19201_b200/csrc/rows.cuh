// Row-wise kernels between the GEMMs: embedding lookup, residual add + RMSNorm, rotary
// embedding + KV-cache append, SiLU gating, per-row top-k with log-sum-exp.
// Model definition (pre-norm blocks, RMSNorm, half-split rotary pairs, gated SiLU MLP) is the
// reading taken for the architecture details the paper leaves to the target VLMs (Section 4).
#pragma once
#include "common.cuh"

// ---------------------------------------------------------------------------------------
// x[r] = embed[tok[r]] (fp32 residual stream).  tok < 0 leaves a zero row.
template <typename T>
__global__ void k_embed(const T *__restrict__ embed, const int *__restrict__ tok, float *x, int d,
                        int vocab, int *status) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, t = tok[r];
  if (t >= vocab) { if (threadIdx.x == 0) atomicMax(status, DREAM_DEV_BAD_INDEX); t = -1; }
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    x[(long long)r * d + i] = t >= 0 ? to_f(embed[(long long)t * d + i]) : 0.f;
}

// Prompt input rows of the prefill: visual embeddings inside [vis_start, vis_start+v),
// token embeddings elsewhere.  Writes the running residual x and a kept copy x0.
template <typename T>
__global__ void k_build_prompt(const T *__restrict__ embed, const T *__restrict__ visual,
                               const int *__restrict__ ids, int vis_start, int v, float *x,
                               float *x0, int d, int vocab, int *status) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x;
  const T *src;
  if (r >= vis_start && r < vis_start + v) src = visual + (long long)(r - vis_start) * d;
  else {
    int t = ids[r < vis_start ? r : r - v];
    if (t < 0 || t >= vocab) { if (threadIdx.x == 0) atomicMax(status, DREAM_DEV_BAD_INDEX); t = 0; }
    src = embed + (long long)t * d;
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float f = to_f(src[i]);
    x[(long long)r * d + i] = f;
    x0[(long long)r * d + i] = f;
  }
}

// ---------------------------------------------------------------------------------------
// Per row: x += (GEMM output, if any); xn = RMSNorm(x) * gain as the next GEMM's input.
// Optional side outputs of the updated residual: `copy` (fp32; when tap_state is given the
// row is copied only if its sequence's tap layer equals `layer`) and `raw` (element type,
// unnormalised: the memory side of Eq. 1 takes features without a norm).
template <typename T>
__global__ void k_resid_norm(float *x, GemmOut gin, int has_in, const T *__restrict__ gain,
                             float eps, int d, T *xn, float *copy, const int *row_seq,
                             const int *tap_state, int layer, T *raw, XLayout lay) {
  __shared__ float sh[33];
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x;
  float *xr = x + (long long)r * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = xr[i];
    if (has_in) { v += gemm_val(gin, r, i); xr[i] = v; }
    ss += v * v;
  }
  float tot = block_sum(ss, sh);
  float inv = rsqrtf(tot / (float)d + eps);
  bool do_copy = copy != nullptr && (tap_state == nullptr || tap_state[row_seq[r]] == layer);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = xr[i];
    if (do_copy) copy[(long long)r * d + i] = v;
    if (raw) store_split<T>(raw + r * lay.row_stride + i, lay.lo_delta, v);
    if (xn) store_split<T>(xn + r * lay.row_stride + i, lay.lo_delta, v * inv * to_f(gain[i]));
  }
}

// ---------------------------------------------------------------------------------------
// Rotary angle of (position, pair index) = position * theta^(-2i/hd).  The inverse frequencies
// are tabulated once in double; the product is taken in double and reduced to [-pi, pi] before
// the single-precision sincos, so long prefixes lose no phase accuracy.
__global__ void k_rope_table(double *inv_freq, int hd, float theta) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < hd / 2) inv_freq[i] = exp2(-2.0 * (double)i / (double)hd * log2((double)theta));
}
__device__ __forceinline__ void rope_cs(int pos, double inv, float *c, float *s) {
  double a = (double)pos * inv;
  const double two_pi = 6.283185307179586476925286766559;
  a -= two_pi * rint(a / two_pi);
  sincosf((float)a, s, c);
}

// Where a row's K/V go.  Target cache: pages [layer][2][page][H_kv][page_tokens][hd].
struct PagedKV {
  void *base;                    // this layer's K pool; V pool = base + kv_stride elements
  long long kv_stride;           // elements between the K pool and the V pool of one layer
  const int *page_table;         // [max_batch][pages_per_seq]
  int pages_per_seq, page_tokens, page_shift, hkv, hd;
  __device__ __forceinline__ long long off(int seq, int slot, int kvh) const {
    int pg = page_table[seq * pages_per_seq + (slot >> page_shift)];
    return (((long long)pg * hkv + kvh) * page_tokens + (slot & (page_tokens - 1))) * hd;
  }
};

// After the QKV GEMM of target rows: rotary on q and k at row_pos, q -> qbuf (fp32),
// k, v -> the paged cache at (row_seq, row_slot).  One block per row; a work item is one
// rotary pair (head, i) so that consecutive threads read consecutive GEMM columns.
template <typename T>
__global__ void k_qkv_post_target(GemmOut g, const int *__restrict__ row_seq,
                                  const int *__restrict__ row_pos, const int *__restrict__ row_slot,
                                  int row0, float *qbuf, PagedKV kv, int H, const double *__restrict__ inv_freq) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int hd = kv.hd, half = hd >> 1, Hkv = kv.hkv;
  int seq = row_seq[r], pos = row_pos[r], slot = row_slot[r];
  T *Kp = (T *)kv.base, *Vp = (T *)kv.base + kv.kv_stride;
  int items = (H + 2 * Hkv) * half;
  for (int w = threadIdx.x; w < items; w += blockDim.x) {
    int hh = w / half, i = w - hh * half;
    float a = gemm_val(g, lr, hh * hd + i), b = gemm_val(g, lr, hh * hd + i + half);
    if (hh < H + Hkv) {
      float c, s;
      rope_cs(pos, inv_freq[i], &c, &s);
      float ra = a * c - b * s, rb = b * c + a * s;
      if (hh < H) {
        float *q = qbuf + ((long long)r * H + hh) * hd;
        q[i] = ra; q[i + half] = rb;
      } else {
        long long o = kv.off(seq, slot, hh - H);
        Kp[o + i] = from_f<T>(ra); Kp[o + i + half] = from_f<T>(rb);
      }
    } else {
      long long o = kv.off(seq, slot, hh - H - Hkv);
      Vp[o + i] = from_f<T>(a); Vp[o + i + half] = from_f<T>(b);
    }
  }
}

// Draft caches are flat per sequence, always fp32 (they are small): [seq][2][H_kv][cap][hd].
struct FlatKV {
  float *base;
  int cap, hkv, hd;
  __device__ __forceinline__ long long off(int seq, int kv, int kvh, int row) const {
    return ((((long long)seq * 2 + kv) * hkv + kvh) * cap + row) * hd;
  }
};

// After a draft QKV GEMM (has_q: the GEMM produced q columns first, then K, then V; otherwise
// K then V only): rotary, q -> qbuf (when has_q), k/v -> draft self-attention cache row
// row_dst[r] (skipped when < 0).  Work items as in k_qkv_post_target.
__global__ void k_qkv_post_draft(GemmOut g, const int *__restrict__ row_seq,
                                 const int *__restrict__ row_pos, const int *__restrict__ row_dst,
                                 int row0, int has_q, float *qbuf, FlatKV kv, int H, const double *__restrict__ inv_freq) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int dst = row_dst[r];
  int hd = kv.hd, half = hd >> 1, Hkv = kv.hkv;
  int seq = row_seq[r], pos = row_pos[r];
  int Hq = has_q ? H : 0;
  float *base = kv.base;
  int items = (Hq + 2 * Hkv) * half;
  for (int w = threadIdx.x; w < items; w += blockDim.x) {
    int hh = w / half, i = w - hh * half;
    if (hh >= Hq && dst < 0) continue;
    float a = gemm_val(g, lr, hh * hd + i), b = gemm_val(g, lr, hh * hd + i + half);
    if (hh < Hq + Hkv) {
      float c, s;
      rope_cs(pos, inv_freq[i], &c, &s);
      float ra = a * c - b * s, rb = b * c + a * s;
      if (hh < Hq) {
        float *q = qbuf + ((long long)r * H + hh) * hd;
        q[i] = ra; q[i + half] = rb;
      } else {
        long long o = kv.off(seq, 0, hh - Hq, dst);
        base[o + i] = ra; base[o + i + half] = rb;
      }
    } else {
      long long o = kv.off(seq, 1, hh - Hq - Hkv, dst);
      base[o + i] = a; base[o + i + half] = b;
    }
  }
}

// Plain copy of a GEMM output [rows][width] into fp32 rows (q of the cross-attention: no rotary)
__global__ void k_gemm_to_f32(GemmOut g, float *dst, int width) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x;
  for (int i = threadIdx.x; i < width; i += blockDim.x) dst[(long long)r * width + i] = gemm_val(g, r, i);
}

// Cross-attention memory rows (Eq. 1: K = S W_K, V = S W_V): GEMM output [rows][2 H_kv hd]
// -> memory cache row of sequence row_seq[r]: row_dst[r] when nperm is null, else the
// tree-region row nperm[seq] + row_in[r].  Negative indices skip the row.
__global__ void k_mem_append(GemmOut g, const int *__restrict__ row_seq,
                             const int *__restrict__ row_dst, const int *__restrict__ row_in,
                             const int *__restrict__ nperm, int row0, FlatKV kv) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int seq = row_seq[r];
  int dst = nperm ? (row_in[r] < 0 ? -1 : nperm[seq] + row_in[r]) : row_dst[r];
  if (dst < 0) return;
  int w = kv.hkv * kv.hd;
  float *base = kv.base;
  for (int i = threadIdx.x; i < w; i += blockDim.x) {
    int h = i / kv.hd, e = i - h * kv.hd;
    base[kv.off(seq, 0, h, dst) + e] = gemm_val(g, lr, i);
    base[kv.off(seq, 1, h, dst) + e] = gemm_val(g, lr, w + i);
  }
}

// act = silu(gate) * up, from a GEMM output whose columns are [gate(ff) | up(ff)].
template <typename T>
__global__ void k_silu_mul(GemmOut g, T *act, int ff, XLayout lay) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.y;
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= ff) return;
  float a = gemm_val(g, r, i), b = gemm_val(g, r, ff + i);
  store_split<T>(act + r * lay.row_stride + i, lay.lo_delta, a / (1.f + __expf(-a)) * b);
}

// x += GEMM output; optional fp32 copy into a per-layer store (prefill tap candidates).
__global__ void k_resid_add(float *x, GemmOut g, int d, float *copy) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = x[(long long)r * d + i] + gemm_val(g, r, i);
    x[(long long)r * d + i] = v;
    if (copy) copy[(long long)r * d + i] = v;
  }
}

// Gather fp32 rows into element-type GEMM input rows: dst[r] = src[idx[r]] (idx < 0 -> zeros).
template <typename T>
__global__ void k_gather_rows(const float *__restrict__ src, const int *__restrict__ idx, T *dst,
                              int d, const int *layer_ptr, int layer_lo, long long layer_stride,
                              XLayout lay) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, s = idx[r];
  if (layer_ptr) src += (long long)(*layer_ptr - layer_lo) * layer_stride;
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    store_split<T>(dst + r * lay.row_stride + i, lay.lo_delta, s >= 0 ? src[(long long)s * d + i] : 0.f);
}

// ---------------------------------------------------------------------------------------
// Per row of a [rows][V] GEMM output: the KTOP largest logits (ties -> lower id), in
// descending order, and the log-sum-exp of the row.  One block per row.
#define TOPK_MAX 16
#define TOPK_THREADS 256
__global__ void __launch_bounds__(TOPK_THREADS)
k_topk_lse(GemmOut g, int V, int ktop, float *top_val, int *top_id, float *lse, float *logits_out) {
  __shared__ float sv[TOPK_THREADS * TOPK_MAX];
  __shared__ int si[TOPK_THREADS * TOPK_MAX];
  __shared__ float red[33];
  __shared__ float cand_v[TOPK_THREADS / 32];
  __shared__ int cand_i[TOPK_THREADS / 32], cand_t[TOPK_THREADS / 32];
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, tid = threadIdx.x;
  float lv[TOPK_MAX];
  int li[TOPK_MAX];
  for (int j = 0; j < TOPK_MAX; ++j) { lv[j] = -INFINITY; li[j] = 0x7fffffff; }
  float m = -INFINITY, z = 0.f;
  for (int c = tid; c < V; c += TOPK_THREADS) {
    float v = gemm_val(g, r, c);
    if (logits_out) logits_out[(long long)r * V + c] = v;
    if (v > m) { z = z * __expf(m - v) + 1.f; m = v; } else z += __expf(v - m);
    if (better(v, c, lv[ktop - 1], li[ktop - 1])) {
      int j = ktop - 1;
      while (j > 0 && better(v, c, lv[j - 1], li[j - 1])) { lv[j] = lv[j - 1]; li[j] = li[j - 1]; --j; }
      lv[j] = v; li[j] = c;
    }
  }
  // log-sum-exp: combine (m, z) pairs in a fixed order
  float bm = m;
  bm = warp_max(bm);
  __syncthreads();
  if ((tid & 31) == 0) red[tid >> 5] = bm;
  __syncthreads();
  if (tid < 32) { float t = tid < TOPK_THREADS / 32 ? red[tid] : -INFINITY; t = warp_max(t); if (tid == 0) red[32] = t; }
  __syncthreads();
  float gm = red[32];
  float tot = block_sum(m == -INFINITY ? 0.f : z * __expf(m - gm), red);
  if (tid == 0) lse[r] = gm + logf(tot);
  // merge the per-thread sorted lists: ktop rounds of a block-wide "best head" selection
  for (int j = 0; j < ktop; ++j) { sv[tid * TOPK_MAX + j] = lv[j]; si[tid * TOPK_MAX + j] = li[j]; }
  int head = 0;
  __syncthreads();
  for (int round = 0; round < ktop; ++round) {
    float v = head < ktop ? sv[tid * TOPK_MAX + head] : -INFINITY;
    int id = head < ktop ? si[tid * TOPK_MAX + head] : 0x7fffffff;
    int t = tid;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, v, o);
      int oi = __shfl_xor_sync(0xffffffffu, id, o), ot = __shfl_xor_sync(0xffffffffu, t, o);
      if (better(ov, oi, v, id)) { v = ov; id = oi; t = ot; }
    }
    if ((tid & 31) == 0) { cand_v[tid >> 5] = v; cand_i[tid >> 5] = id; cand_t[tid >> 5] = t; }
    __syncthreads();
    float bv = cand_v[0]; int bi = cand_i[0], bt = cand_t[0];
    for (int w = 1; w < TOPK_THREADS / 32; ++w)
      if (better(cand_v[w], cand_i[w], bv, bi)) { bv = cand_v[w]; bi = cand_i[w]; bt = cand_t[w]; }
    if (tid == bt) ++head;
    if (tid == 0) { top_val[r * ktop + round] = bv; top_id[r * ktop + round] = bi; }
    __syncthreads();
  }
}
