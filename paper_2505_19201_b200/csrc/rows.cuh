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
#define NORM_THREADS 512
#define NORM_NV 4                // float4 groups a thread keeps in registers (rows up to 8192 wide)
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS)
k_resid_norm(float *x, GemmOut gin, int has_in, const T *__restrict__ gain,
             float eps, int d, T *xn, float *copy, const int *row_seq,
             const int *tap_state, int layer, T *raw, XLayout lay) {
  __shared__ float sh[33];
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, d4 = d >> 2;
  float *xr = x + (long long)r * d;
  float4 v[NORM_NV];
  float ss = 0.f;
  // every load of the row is issued before the first use
#pragma unroll
  for (int j = 0; j < NORM_NV; ++j) {
    int i = threadIdx.x + j * NORM_THREADS;
    v[j] = i < d4 ? ld_f4(xr + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (has_in) {
    float4 gv[NORM_NV];
#pragma unroll
    for (int j = 0; j < NORM_NV; ++j) {
      int i = threadIdx.x + j * NORM_THREADS;
      gv[j] = i < d4 ? gemm_val4(gin, r, 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < NORM_NV; ++j) {
      int i = threadIdx.x + j * NORM_THREADS;
      v[j].x += gv[j].x; v[j].y += gv[j].y; v[j].z += gv[j].z; v[j].w += gv[j].w;
      if (i < d4) *reinterpret_cast<float4 *>(xr + 4 * i) = v[j];
    }
  }
#pragma unroll
  for (int j = 0; j < NORM_NV; ++j) ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
  for (int i = threadIdx.x + NORM_NV * NORM_THREADS; i < d4; i += NORM_THREADS) {      // rows wider than 8192
    float4 t = ld_f4(xr + 4 * i);
    if (has_in) {
      float4 gq = gemm_val4(gin, r, 4 * i);
      t.x += gq.x; t.y += gq.y; t.z += gq.z; t.w += gq.w;
      *reinterpret_cast<float4 *>(xr + 4 * i) = t;
    }
    ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
  }
  float tot = block_sum(ss, sh);
  float inv = rsqrtf(tot / (float)d + eps);
  bool do_copy = copy != nullptr && (tap_state == nullptr || tap_state[row_seq[r]] == layer);
  auto emit = [&](int i, float4 t) {
    if (do_copy) *reinterpret_cast<float4 *>(copy + (long long)r * d + 4 * i) = t;
    if (raw) store_split4<T>(raw + r * lay.row_stride + 4 * i, lay.lo_delta, t);
    if (xn) {
      float4 gq = ld_f4(gain + 4 * i);
      store_split4<T>(xn + r * lay.row_stride + 4 * i, lay.lo_delta,
                      make_float4(t.x * inv * gq.x, t.y * inv * gq.y, t.z * inv * gq.z, t.w * inv * gq.w));
    }
  };
#pragma unroll
  for (int j = 0; j < NORM_NV; ++j) {
    int i = threadIdx.x + j * NORM_THREADS;
    if (i < d4) emit(i, v[j]);
  }
  for (int i = threadIdx.x + NORM_NV * NORM_THREADS; i < d4; i += NORM_THREADS) emit(i, ld_f4(xr + 4 * i));
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
// k, v -> the paged cache at (row_seq, row_slot).  grid (rows, ceil(items / 256)); a work item
// is four neighbouring rotary pairs of one head, read and written as 128-bit words.
template <typename T>
__global__ void k_qkv_post_target(GemmOut g, const int *__restrict__ row_seq,
                                  const int *__restrict__ row_pos, const int *__restrict__ row_slot,
                                  int row0, void *qbuf, PagedKV kv, int H, const double *__restrict__ inv_freq) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int hd = kv.hd, half = hd >> 1, q4 = half >> 2, Hkv = kv.hkv;
  int w = blockIdx.y * blockDim.x + threadIdx.x;
  if (w >= (H + 2 * Hkv) * q4) return;
  int hh = w / q4, i = (w - hh * q4) * 4;
  int seq = row_seq[r], pos = row_pos[r], slot = row_slot[r];
  T *Kp = (T *)kv.base, *Vp = (T *)kv.base + kv.kv_stride;
  float4 a = gemm_val4(g, lr, hh * hd + i), b = gemm_val4(g, lr, hh * hd + i + half);
  if (hh < H + Hkv) {
    float c0, s0, c1, s1, c2, s2, c3, s3;
    rope_cs(pos, inv_freq[i], &c0, &s0); rope_cs(pos, inv_freq[i + 1], &c1, &s1);
    rope_cs(pos, inv_freq[i + 2], &c2, &s2); rope_cs(pos, inv_freq[i + 3], &c3, &s3);
    float4 ra = make_float4(a.x * c0 - b.x * s0, a.y * c1 - b.y * s1, a.z * c2 - b.z * s2, a.w * c3 - b.w * s3);
    float4 rb = make_float4(b.x * c0 + a.x * s0, b.y * c1 + a.y * s1, b.z * c2 + a.z * s2, b.w * c3 + a.w * s3);
    if (hh < H) {
      q_store4(qbuf, sizeof(T) == 2, (long long)r * H + hh, hd, i, ra);
      q_store4(qbuf, sizeof(T) == 2, (long long)r * H + hh, hd, i + half, rb);
    } else {
      long long o = kv.off(seq, slot, hh - H);
      store_split4<T>(Kp + o + i, 0, ra);
      store_split4<T>(Kp + o + i + half, 0, rb);
    }
  } else {
    long long o = kv.off(seq, slot, hh - H - Hkv);
    store_split4<T>(Vp + o + i, 0, a);
    store_split4<T>(Vp + o + i + half, 0, b);
  }
}

// Draft caches are flat per sequence and hold 4 bytes per element (they are small):
// [seq][2][H_kv][cap] rows of hd floats (fp32 configurations), or of 2 * hd bf16 = a high row
// then a low row (bf16 configurations: what the tensor-core attention reads directly).
struct FlatKV {
  void *base;
  int cap, hkv, hd, split;
  __device__ __forceinline__ long long off(int seq, int kv, int kvh, int row) const {
    return ((((long long)seq * 2 + kv) * hkv + kvh) * cap + row) * (split ? 2 : 1) * hd;
  }
  __device__ __forceinline__ void store4(long long o, int e, float4 v) const {
    if (split) store_split4<bf16>((bf16 *)base + o + e, hd, v);
    else *reinterpret_cast<float4 *>((float *)base + o + e) = v;
  }
};

// After a draft QKV GEMM (has_q: the GEMM produced q columns first, then K, then V; otherwise
// K then V only): rotary, q -> qbuf (when has_q), k/v -> draft self-attention cache row
// row_dst[r] (skipped when < 0).  Work items and grid as in k_qkv_post_target.
__global__ void k_qkv_post_draft(GemmOut g, const int *__restrict__ row_seq,
                                 const int *__restrict__ row_pos, const int *__restrict__ row_dst,
                                 int row0, int has_q, void *qbuf, FlatKV kv, int H, const double *__restrict__ inv_freq) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int hd = kv.hd, half = hd >> 1, q4 = half >> 2, Hkv = kv.hkv;
  int Hq = has_q ? H : 0;
  int w = blockIdx.y * blockDim.x + threadIdx.x;
  if (w >= (Hq + 2 * Hkv) * q4) return;
  int hh = w / q4, i = (w - hh * q4) * 4;
  int dst = row_dst[r], seq = row_seq[r], pos = row_pos[r];
  if (hh >= Hq && dst < 0) return;
  float4 a = gemm_val4(g, lr, hh * hd + i), b = gemm_val4(g, lr, hh * hd + i + half);
  if (hh < Hq + Hkv) {
    float c0, s0, c1, s1, c2, s2, c3, s3;
    rope_cs(pos, inv_freq[i], &c0, &s0); rope_cs(pos, inv_freq[i + 1], &c1, &s1);
    rope_cs(pos, inv_freq[i + 2], &c2, &s2); rope_cs(pos, inv_freq[i + 3], &c3, &s3);
    float4 ra = make_float4(a.x * c0 - b.x * s0, a.y * c1 - b.y * s1, a.z * c2 - b.z * s2, a.w * c3 - b.w * s3);
    float4 rb = make_float4(b.x * c0 + a.x * s0, b.y * c1 + a.y * s1, b.z * c2 + a.z * s2, b.w * c3 + a.w * s3);
    if (hh < Hq) {
      q_store4(qbuf, kv.split, (long long)r * H + hh, hd, i, ra);
      q_store4(qbuf, kv.split, (long long)r * H + hh, hd, i + half, rb);
    } else {
      long long o = kv.off(seq, 0, hh - Hq, dst);
      kv.store4(o, i, ra);
      kv.store4(o, i + half, rb);
    }
  } else {
    long long o = kv.off(seq, 1, hh - Hq - Hkv, dst);
    kv.store4(o, i, a);
    kv.store4(o, i + half, b);
  }
}

// A GEMM output [rows][H * hd] becomes the query rows of the cross-attention (no rotary).
// grid (rows, ceil(H * hd / 1024)).
__global__ void k_gemm_to_q(GemmOut g, void *qbuf, int H, int hd, int split) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, i = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  if (i >= H * hd) return;
  int h = i / hd;
  q_store4(qbuf, split, (long long)r * H + h, hd, i - h * hd, gemm_val4(g, r, i));
}

// Cross-attention memory rows (Eq. 1: K = S W_K, V = S W_V): GEMM output [rows][2 H_kv hd]
// -> memory cache row of sequence row_seq[r]: row_dst[r] when nperm is null, else the
// tree-region row nperm[seq] + row_in[r].  Negative indices skip the row.
// grid (rows, ceil(2 H_kv hd / 1024)).
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
  int i = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  if (i >= 2 * w) return;
  int which = i >= w ? 1 : 0, j = i - which * w;
  int h = j / kv.hd, e = j - h * kv.hd;
  kv.store4(kv.off(seq, which, h, dst), e, gemm_val4(g, lr, i));
}

// act = silu(gate) * up, from a GEMM output whose columns are [gate(ff) | up(ff)].
// grid (ceil(ff / 1024), rows).
template <typename T>
__global__ void k_silu_mul(GemmOut g, T *act, int ff, XLayout lay) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.y;
  int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= ff) return;
  float4 a = gemm_val4(g, r, i), b = gemm_val4(g, r, ff + i);
  float4 o = make_float4(a.x / (1.f + __expf(-a.x)) * b.x, a.y / (1.f + __expf(-a.y)) * b.y,
                         a.z / (1.f + __expf(-a.z)) * b.z, a.w / (1.f + __expf(-a.w)) * b.w);
  store_split4<T>(act + r * lay.row_stride + i, lay.lo_delta, o);
}

// x += GEMM output; optional fp32 copy into a per-layer store (prefill tap candidates).
// grid (rows, ceil(d / 1024)).
__global__ void k_resid_add(float *x, GemmOut g, int d, float *copy) {
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, i = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  if (i >= d) return;
  float4 v = ld_f4(x + (long long)r * d + i), t = gemm_val4(g, r, i);
  v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
  *reinterpret_cast<float4 *>(x + (long long)r * d + i) = v;
  if (copy) *reinterpret_cast<float4 *>(copy + (long long)r * d + i) = v;
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
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4)
    store_split4<T>(dst + r * lay.row_stride + i, lay.lo_delta,
                    s >= 0 ? ld_f4(src + (long long)s * d + i) : make_float4(0.f, 0.f, 0.f, 0.f));
}

// ---------------------------------------------------------------------------------------
// Per row of a [rows][V] GEMM output: the KTOP largest logits (ties -> lower id), in
// descending order, and the log-sum-exp of the row.  grid (rows, nsplit): block (r, sp) scans
// columns [sp * TOPK_COLS, (sp + 1) * TOPK_COLS) and leaves a sorted partial list and an (m, z)
// pair; the block that finishes a row last merges the partials, always in the same order.
#define TOPK_MAX 16
#define TOPK_THREADS 256
#define TOPK_COLS 4096
struct TopkScratch {
  float *pv;       // [rows][nsplit][TOPK_MAX] partial values
  int *pi;         // [rows][nsplit][TOPK_MAX] partial ids
  float *pm, *pz;  // [rows][nsplit] running max and sum of exp
  int *counter;    // [rows] blocks done; zero between launches
};

// Block-wide selection of the `ktop` best heads of per-thread sorted lists kept in shared memory
// (list t = sv/si[t * TOPK_MAX ..], `len` valid entries for t < nlists).  Round j's winner goes
// to out_v/out_i[j].
__device__ __forceinline__ void topk_merge_lists(const float *sv, const int *si, int nlists, int len, int ktop,
                                                 float *out_v, int *out_i, float *cand_v, int *cand_i, int *cand_t) {
  int tid = threadIdx.x, head = 0;
  for (int round = 0; round < ktop; ++round) {
    bool live = tid < nlists && head < len;
    float v = live ? sv[tid * TOPK_MAX + head] : -INFINITY;
    int id = live ? si[tid * TOPK_MAX + head] : 0x7fffffff;
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
    if (tid == 0) { out_v[round] = bv; out_i[round] = bi; }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(TOPK_THREADS)
k_topk_lse(GemmOut g, int V, int ktop, int nsplit, TopkScratch ts, float *top_val, int *top_id, float *lse,
           float *logits_out) {
  __shared__ float sv[TOPK_THREADS * TOPK_MAX];
  __shared__ int si[TOPK_THREADS * TOPK_MAX];
  __shared__ float red[33];
  __shared__ float cand_v[TOPK_THREADS / 32];
  __shared__ int cand_i[TOPK_THREADS / 32], cand_t[TOPK_THREADS / 32];
  __shared__ int is_last;
  pdl_trigger();
  pdl_wait();
  int r = blockIdx.x, sp = blockIdx.y, tid = threadIdx.x;
  int c0 = sp * TOPK_COLS, c1 = min(V, c0 + TOPK_COLS);
  float lv[TOPK_MAX];
  int li[TOPK_MAX];
  for (int j = 0; j < TOPK_MAX; ++j) { lv[j] = -INFINITY; li[j] = 0x7fffffff; }
  float m = -INFINITY, z = 0.f;
  auto consider = [&](float v, int c) {
    if (v > m) { z = z * __expf(m - v) + 1.f; m = v; } else z += __expf(v - m);
    if (better(v, c, lv[ktop - 1], li[ktop - 1])) {
      int j = ktop - 1;
      while (j > 0 && better(v, c, lv[j - 1], li[j - 1])) { lv[j] = lv[j - 1]; li[j] = li[j - 1]; --j; }
      lv[j] = v; li[j] = c;
    }
  };
  if ((V & 3) == 0) {
    for (int c = c0 + tid * 4; c < c1; c += TOPK_THREADS * 4) {
      float4 v = gemm_val4(g, r, c);
      if (logits_out) *reinterpret_cast<float4 *>(logits_out + (long long)r * V + c) = v;
      consider(v.x, c); consider(v.y, c + 1); consider(v.z, c + 2); consider(v.w, c + 3);
    }
  } else {
    for (int c = c0 + tid; c < c1; c += TOPK_THREADS) {
      float v = gemm_val(g, r, c);
      if (logits_out) logits_out[(long long)r * V + c] = v;
      consider(v, c);
    }
  }
  // (m, z) of this block's columns, combined in a fixed order
  float bm = warp_max(m);
  __syncthreads();
  if ((tid & 31) == 0) red[tid >> 5] = bm;
  __syncthreads();
  if (tid < 32) { float t = tid < TOPK_THREADS / 32 ? red[tid] : -INFINITY; t = warp_max(t); if (tid == 0) red[32] = t; }
  __syncthreads();
  float gm = red[32];
  float tot = block_sum(m == -INFINITY ? 0.f : z * __expf(m - gm), red);
  long long po = (long long)r * nsplit + sp;
  if (tid == 0) { ts.pm[po] = gm; ts.pz[po] = tot; }
  // this block's sorted top-ktop
  for (int j = 0; j < ktop; ++j) { sv[tid * TOPK_MAX + j] = lv[j]; si[tid * TOPK_MAX + j] = li[j]; }
  __syncthreads();
  topk_merge_lists(sv, si, TOPK_THREADS, ktop, ktop, ts.pv + po * TOPK_MAX, ts.pi + po * TOPK_MAX, cand_v, cand_i, cand_t);
  // the last block of the row merges
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    int old = atomicAdd(ts.counter + r, 1);
    is_last = old == nsplit - 1;
    if (is_last) ts.counter[r] = 0;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  if (tid < nsplit) {
    for (int j = 0; j < ktop; ++j) {
      sv[tid * TOPK_MAX + j] = __ldcg(ts.pv + ((long long)r * nsplit + tid) * TOPK_MAX + j);
      si[tid * TOPK_MAX + j] = __ldcg(ts.pi + ((long long)r * nsplit + tid) * TOPK_MAX + j);
    }
  }
  if (tid == 0) {
    float mm = -INFINITY, zz = 0.f;
    for (int q = 0; q < nsplit; ++q) mm = fmaxf(mm, __ldcg(ts.pm + (long long)r * nsplit + q));
    for (int q = 0; q < nsplit; ++q) zz += __ldcg(ts.pz + (long long)r * nsplit + q) * __expf(__ldcg(ts.pm + (long long)r * nsplit + q) - mm);
    lse[r] = mm + logf(zz);
  }
  __syncthreads();
  topk_merge_lists(sv, si, nsplit, ktop, ktop, top_val + (long long)r * ktop, top_id + (long long)r * ktop, cand_v, cand_i, cand_t);
}
