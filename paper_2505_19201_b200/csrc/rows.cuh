// Row-wise kernels between the GEMMs: embedding lookup, residual add + RMSNorm, rotary
// embedding + KV-cache append, SiLU gating, per-row top-k with log-sum-exp.
// Model definition (pre-norm blocks, RMSNorm, half-split rotary pairs, gated SiLU MLP) is the
// reading taken for the architecture details the paper leaves to the target VLMs (Section 4).
#pragma once
#include "common.cuh"

// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void rope_cs(int pos, double inv, float *c, float *s);
// x[r] = embed[tok[r]] (fp32 residual stream).  tok < 0 leaves a zero row.  One thread per four
// elements: grid (rows, ceil(d / 1024)).  With rope_tab the first block of a row also tabulates
// the row's rotary factors for every layer of the call: rope_tab[r][i] = (cos, sin)(pos[r] *
// inv_freq[i]), i < half.
template <typename T>
__global__ void k_embed(const T *__restrict__ embed, const int *__restrict__ tok, float *x, int d,
                        int vocab, int *status, const int *__restrict__ pos, const double *__restrict__ inv_freq,
                        float2 *rope_tab, int half) {
  kernel_entry(TR_k_embed);
  int r = blockIdx.x, t = tok[r];
  if (rope_tab && blockIdx.y == 0)
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
      float c, s;
      rope_cs(pos[r], inv_freq[i], &c, &s);
      rope_tab[(long long)r * half + i] = make_float2(c, s);
    }
  int i = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  if (t >= vocab) { if (threadIdx.x == 0 && blockIdx.y == 0) atomicMax(status, DREAM_DEV_BAD_INDEX); t = -1; }
  if (i >= d) return;
  *reinterpret_cast<float4 *>(x + (long long)r * d + i) = t >= 0 ? ld_f4(embed + (long long)t * d + i) : make_float4(0.f, 0.f, 0.f, 0.f);
}

// Prompt input rows of the prefill: visual embeddings inside [vis_start, vis_start+v),
// token embeddings elsewhere.  Writes the running residual x and a kept copy x0.
template <typename T>
__global__ void k_build_prompt(const T *__restrict__ embed, const T *__restrict__ visual,
                               const int *__restrict__ ids, int vis_start, int v, float *x,
                               float *x0, int d, int vocab, int *status) {
  kernel_entry(TR_k_build_prompt);
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
// Block size: ceil(d / 4 / NV) threads rounded up to a warp (at most 1024); a thread keeps NV
// groups of four elements, so rows of up to 4096 * NV elements fit.  The partial-sum slots of a
// value are all fetched at once (up to 12 per round trip).
template <typename T, int NV>
__global__ void __launch_bounds__(1024)
k_resid_norm(float *x, GemmOut gin, int has_in, const T *__restrict__ gain,
             float eps, int d, T *xn, float *copy, const int *row_seq,
             const int *tap_state, int layer, T *raw, XLayout lay) {
  __shared__ float sh[33];
  const int r = blockIdx.x, d4 = d >> 2, nt = blockDim.x;
  // the gains are weights: they can be fetched before the predecessor has finished
  float4 gq[NV];
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = threadIdx.x + j * nt;
    gq[j] = (xn && i < d4) ? ld_f4(gain + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  kernel_entry(TR_k_resid_norm);
  float *xr = x + (long long)r * d;
  float4 v[NV];
  float ss = 0.f;
  // every load of the row is issued before the first use
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = threadIdx.x + j * nt;
    v[j] = i < d4 ? ld_f4(xr + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (has_in) {
    float4 gv[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int i = threadIdx.x + j * nt;
      gv[j] = i < d4 ? gemm_val4_wide<12 / NV>(gin, r, 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int i = threadIdx.x + j * nt;
      v[j].x += gv[j].x; v[j].y += gv[j].y; v[j].z += gv[j].z; v[j].w += gv[j].w;
      if (i < d4) *reinterpret_cast<float4 *>(xr + 4 * i) = v[j];
    }
  }
#pragma unroll
  for (int j = 0; j < NV; ++j) ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
  float tot = block_sum(ss, sh);
  float inv = rsqrtf(tot / (float)d + eps);
  bool do_copy = copy != nullptr && (tap_state == nullptr || tap_state[row_seq[r]] == layer);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = threadIdx.x + j * nt;
    if (i >= d4) continue;
    float4 t = v[j];
    if (do_copy) *reinterpret_cast<float4 *>(copy + (long long)r * d + 4 * i) = t;
    if (raw) store_split4<T>(raw + r * lay.row_stride + 4 * i, lay.lo_delta, t);
    if (xn)
      store_split4<T>(xn + r * lay.row_stride + 4 * i, lay.lo_delta,
                      make_float4(t.x * inv * gq[j].x, t.y * inv * gq[j].y, t.z * inv * gq[j].z, t.w * inv * gq[j].w));
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

// (cos, sin) of four neighbouring rotary indices i..i+3 (i a multiple of 4) of row r: from the
// table k_embed made for the call's rows, or computed when there is none (prefill).
__device__ __forceinline__ void rope_cs4(const float2 *tab, int r, int half, int pos, const double *inv_freq, int i,
                                         float4 &cs01, float4 &cs23) {
  if (tab) {
    const float4 *t = reinterpret_cast<const float4 *>(tab + (long long)r * half + i);
    cs01 = t[0]; cs23 = t[1];
  } else {
    rope_cs(pos, inv_freq[i], &cs01.x, &cs01.y); rope_cs(pos, inv_freq[i + 1], &cs01.z, &cs01.w);
    rope_cs(pos, inv_freq[i + 2], &cs23.x, &cs23.y); rope_cs(pos, inv_freq[i + 3], &cs23.z, &cs23.w);
  }
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
                                  int row0, void *qbuf, PagedKV kv, int H, const double *__restrict__ inv_freq,
                                  const float2 *__restrict__ rope_tab) {
  kernel_entry(TR_k_qkv_post_target);
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int hd = kv.hd, half = hd >> 1, q4 = half >> 2, Hkv = kv.hkv;
  int w = blockIdx.y * blockDim.x + threadIdx.x;
  if (w >= (H + 2 * Hkv) * q4) return;
  int hh = w / q4, i = (w - hh * q4) * 4;
  int seq = row_seq[r], pos = row_pos[r], slot = row_slot[r];
  if (hh >= H && slot < 0) return;                 // an idle row (malformed tree node) stores no K/V
  T *Kp = (T *)kv.base, *Vp = (T *)kv.base + kv.kv_stride;
  float4 cs01 = make_float4(1.f, 0.f, 1.f, 0.f), cs23 = cs01;
  if (hh < H + Hkv) rope_cs4(rope_tab, r, half, pos, inv_freq, i, cs01, cs23);      // fetched along with the slots
  float4 a = gemm_val4_wide<4>(g, lr, hh * hd + i), b = gemm_val4_wide<4>(g, lr, hh * hd + i + half);
  if (hh < H + Hkv) {
    const float c0 = cs01.x, s0 = cs01.y, c1 = cs01.z, s1 = cs01.w, c2 = cs23.x, s2 = cs23.y, c3 = cs23.z, s3 = cs23.w;
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
                                 int row0, int has_q, void *qbuf, FlatKV kv, int H, const double *__restrict__ inv_freq,
                                 const float2 *__restrict__ rope_tab) {
  kernel_entry(TR_k_qkv_post_draft);
  int r = blockIdx.x + row0, lr = blockIdx.x;
  int hd = kv.hd, half = hd >> 1, q4 = half >> 2, Hkv = kv.hkv;
  int Hq = has_q ? H : 0;
  int w = blockIdx.y * blockDim.x + threadIdx.x;
  if (w >= (Hq + 2 * Hkv) * q4) return;
  int hh = w / q4, i = (w - hh * q4) * 4;
  int dst = row_dst[r], seq = row_seq[r], pos = row_pos[r];
  if (hh >= Hq && dst < 0) return;
  float4 cs01 = make_float4(1.f, 0.f, 1.f, 0.f), cs23 = cs01;
  if (hh < Hq + Hkv) rope_cs4(rope_tab, r, half, pos, inv_freq, i, cs01, cs23);
  float4 a = gemm_val4_wide<4>(g, lr, hh * hd + i), b = gemm_val4_wide<4>(g, lr, hh * hd + i + half);
  if (hh < Hq + Hkv) {
    const float c0 = cs01.x, s0 = cs01.y, c1 = cs01.z, s1 = cs01.w, c2 = cs23.x, s2 = cs23.y, c3 = cs23.z, s3 = cs23.w;
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
  kernel_entry(TR_k_gemm_to_q);
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
  kernel_entry(TR_k_mem_append);
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
  kernel_entry(TR_k_silu_mul);
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
  kernel_entry(TR_k_resid_add);
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
  kernel_entry(TR_k_gather_rows);
  int r = blockIdx.x, s = idx[r];
  if (layer_ptr) src += (long long)(*layer_ptr - layer_lo) * layer_stride;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4)
    store_split4<T>(dst + r * lay.row_stride + i, lay.lo_delta,
                    s >= 0 ? ld_f4(src + (long long)s * d + i) : make_float4(0.f, 0.f, 0.f, 0.f));
}

// ---------------------------------------------------------------------------------------
// Per row of a [rows][V] GEMM output: the KTOP largest logits (ties -> lower id), in
// descending order, and the log-sum-exp of the row.  grid (rows, nsplit): block (r, sp) scans
// columns [sp * NV * 256, (sp + 1) * NV * 256), NV (4 or 16) per thread held in registers, and leaves a
// sorted partial list and an (m, z) pair; the block that finishes a row last merges the partials,
// always in the same order.  Selection is KTOP rounds of a block-wide "best remaining" search.
#define TOPK_MAX 16
#define TOPK_THREADS 256
#define TOPK_COLS 4096
#define TOPK_PER_THREAD (TOPK_COLS / TOPK_THREADS)
struct TopkScratch {
  float *pv;       // [rows][nsplit][TOPK_MAX] partial values
  int *pi;         // [rows][nsplit][TOPK_MAX] partial ids
  float *pm, *pz;  // [rows][nsplit] running max and sum of exp
  int *counter;    // [rows] blocks done; zero between launches
};

// The ktop best of a block's candidates (NV per thread, in registers), in order, to out_v/out_i.
// Two levels, so that only one block-wide step is needed: every warp selects its own ktop best in
// ktop rounds of "best remaining" (a scan of the thread's candidates and a warp reduction), then
// warp 0 selects from the warps' lists the same way.  Ids are unique, so a winner has one owner.
// sh_* hold TOPK_THREADS / 32 * TOPK_MAX entries.
template <int NV>
__device__ __forceinline__ void topk_round(const float (&v)[NV], const int (&id)[NV], unsigned &taken, float &wv, int &wi) {
  float bv = -INFINITY;
  int bi = 0x7fffffff, bj = -1;
#pragma unroll
  for (int j = 0; j < NV; ++j)
    if (!((taken >> j) & 1u) && better(v[j], id[j], bv, bi)) { bv = v[j]; bi = id[j]; bj = j; }
  wv = bv; wi = bi;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, wv, o);
    int oi = __shfl_xor_sync(0xffffffffu, wi, o);
    if (better(ov, oi, wv, wi)) { wv = ov; wi = oi; }
  }
  if (bj >= 0 && bi == wi && bv == wv) taken |= 1u << bj;
}
template <int NV>
__device__ __forceinline__ void topk_rounds(const float (&v)[NV], const int (&id)[NV], int ktop, float *out_v, int *out_i,
                                            float *sh_v, int *sh_i) {
  constexpr int NW = TOPK_THREADS / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned taken = 0u;
  for (int round = 0; round < ktop; ++round) {
    float wv;
    int wi;
    topk_round<NV>(v, id, taken, wv, wi);
    if (lane == 0) { sh_v[warp * TOPK_MAX + round] = wv; sh_i[warp * TOPK_MAX + round] = wi; }
  }
  __syncthreads();
  if (warp == 0) {
    constexpr int NC = NW * TOPK_MAX / 32;           // candidates per lane
    float cv[NC];
    int ci[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
      int e = j * 32 + lane;
      bool ok = e < NW * ktop;
      int q = ok ? e / ktop : 0, w = ok ? e - q * ktop : 0;
      cv[j] = ok ? sh_v[q * TOPK_MAX + w] : -INFINITY;
      ci[j] = ok ? sh_i[q * TOPK_MAX + w] : 0x7fffffff;
    }
    unsigned tk = 0u;
    for (int round = 0; round < ktop; ++round) {
      float wv;
      int wi;
      topk_round<NC>(cv, ci, tk, wv, wi);
      if (lane == 0) { out_v[round] = wv; out_i[round] = wi; }
    }
  }
  __syncthreads();
}

template <int NV>
__global__ void __launch_bounds__(TOPK_THREADS)
k_topk_lse(GemmOut g, int V, int ktop, int nsplit, TopkScratch ts, float *top_val, int *top_id, float *lse,
           float *logits_out) {
  __shared__ float red[33];
  __shared__ float sh_v[TOPK_THREADS / 32 * TOPK_MAX];
  __shared__ int sh_i[TOPK_THREADS / 32 * TOPK_MAX];
  __shared__ int is_last;
  kernel_entry(TR_k_topk_lse);
  int r = blockIdx.x, sp = blockIdx.y, tid = threadIdx.x;
  int c0 = sp * (NV * TOPK_THREADS);
  float v[NV];
  int id[NV];
  if ((V & 3) == 0) {
    float4 q[NV / 4];
#pragma unroll
    for (int j = 0; j < NV / 4; ++j) {
      int c = c0 + (j * TOPK_THREADS + tid) * 4;
      q[j] = c < V ? gemm_val4(g, r, c) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
#pragma unroll
    for (int j = 0; j < NV / 4; ++j) {
      int c = c0 + (j * TOPK_THREADS + tid) * 4;
      if (logits_out && c < V) *reinterpret_cast<float4 *>(logits_out + (long long)r * V + c) = q[j];
      v[4 * j] = q[j].x; v[4 * j + 1] = q[j].y; v[4 * j + 2] = q[j].z; v[4 * j + 3] = q[j].w;
      id[4 * j] = c; id[4 * j + 1] = c + 1; id[4 * j + 2] = c + 2; id[4 * j + 3] = c + 3;
    }
  } else {
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int c = c0 + j * TOPK_THREADS + tid;
      v[j] = c < V ? gemm_val(g, r, c) : -INFINITY;
      id[j] = c;
      if (logits_out && c < V) logits_out[(long long)r * V + c] = v[j];
    }
  }
#pragma unroll
  for (int j = 0; j < NV; ++j) if (id[j] >= V) id[j] = 0x7fffffff;
  // (m, z) of this block's columns, combined in a fixed order
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < NV; ++j) m = fmaxf(m, v[j]);
  float bm = warp_max(m);
  if ((tid & 31) == 0) red[tid >> 5] = bm;
  __syncthreads();
  if (tid < 32) { float t = tid < TOPK_THREADS / 32 ? red[tid] : -INFINITY; t = warp_max(t); if (tid == 0) red[32] = t; }
  __syncthreads();
  float gm = red[32];
  float z = 0.f;
#pragma unroll
  for (int j = 0; j < NV; ++j) z += __expf(v[j] - gm);        // exp(-inf) = 0 for padding
  float tot = block_sum(z, red);
  long long po = (long long)r * nsplit + sp;
  if (tid == 0) { ts.pm[po] = gm; ts.pz[po] = tot; }
  topk_rounds<NV>(v, id, ktop, ts.pv + po * TOPK_MAX, ts.pi + po * TOPK_MAX, sh_v, sh_i);
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
  // candidates: nsplit lists of ktop entries, up to 4 per thread (nsplit * ktop <= 1024)
  float cv[4];
  int ci[4];
  int ncand = nsplit * ktop;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    int e = j * TOPK_THREADS + tid;
    bool ok = e < ncand;
    int q = ok ? e / ktop : 0, w = ok ? e - q * ktop : 0;
    cv[j] = ok ? __ldcg(ts.pv + ((long long)r * nsplit + q) * TOPK_MAX + w) : -INFINITY;
    ci[j] = ok ? __ldcg(ts.pi + ((long long)r * nsplit + q) * TOPK_MAX + w) : 0x7fffffff;
  }
  if (tid < 32) {                 // log-sum-exp of the row from the blocks' (max, sum) pairs, one warp, fixed order
    float pm[8], pz[8];           // up to 256 blocks
    float mm = -INFINITY;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      int q = k * 32 + tid;
      pm[k] = q < nsplit ? __ldcg(ts.pm + (long long)r * nsplit + q) : -INFINITY;
      pz[k] = q < nsplit ? __ldcg(ts.pz + (long long)r * nsplit + q) : 0.f;
      mm = fmaxf(mm, pm[k]);
    }
    mm = warp_max(mm);
    float zz = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) zz += pz[k] * __expf(pm[k] - mm);         // exp(-inf) = 0 for the padding
    zz = warp_sum(zz);
    if (tid == 0) lse[r] = mm + logf(zz);
  }
  topk_rounds<4>(cv, ci, ktop, top_val + (long long)r * ktop, top_id + (long long)r * ktop, sh_v, sh_i);
}
