// Row-wise work that runs inside the GEMM kernel, ahead of the GEMM whose input it produces:
// residual add + RMSNorm, SiLU gating, and the merge of the attention chunk partials.  The 256
// threads of the GEMM kernel's epilogue warps execute it while the weight ring is already filling,
// so the only cost left on the critical path is the work itself plus one grid-wide barrier
// instead of a kernel boundary.  The same arithmetic, in the same order, as the stand-alone
// kernels k_resid_norm, k_silu_mul and k_attn_combine.
#pragma once
#include "common.cuh"

#define PRO_THREADS 256
#define PRO_NV 8                 // float4 groups a thread keeps of a row (rows up to 8192 wide)

enum { PRO_NONE = 0, PRO_NORM = 1, PRO_SILU = 2, PRO_COMBINE = 3 };

struct ProNorm {                 // x += gin (optional); xn = RMSNorm(x) * gain; side copies
  float *x;
  GemmOut gin;
  int has_in;
  const bf16 *gain;
  float eps;
  int d;
  bf16 *xn;                      // may be null
  float *copy;                   // fp32 copy of the updated row (tap capture), may be null
  const int *row_seq, *tap_state;
  int layer;
  bf16 *raw;                     // unnormalised GEMM input rows, may be null
  XLayout lay;
};
struct ProSilu {                 // act = silu(gate) * up from a [gate | up] GEMM output
  GemmOut g;
  bf16 *act;
  int ff;
  XLayout lay;
};
struct ProCombine {              // attention partials -> attention output rows
  const float *part_o, *part_ml;
  const int *row_in;
  int n_chunks, n_rt, H, G, rows_per_seq, hd;
  bf16 *out;
  XLayout lay;
};
struct Prologue {
  int kind, rows;
  ProNorm norm;
  ProSilu silu;
  ProCombine comb;
};

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int threads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Sum over the PRO_THREADS prologue threads (tid = 0..255), fixed order; sh holds 8 floats.
__device__ __forceinline__ float pro_group_sum(float v, float *sh, int tid) {
  v = warp_sum(v);
  if ((tid & 31) == 0) sh[tid >> 5] = v;
  named_bar_sync(2, PRO_THREADS);
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < PRO_THREADS / 32; ++w) t += sh[w];
  named_bar_sync(2, PRO_THREADS);            // sh may be rewritten by the next row
  return t;
}

__device__ __forceinline__ void pro_norm(const ProNorm &a, int rows, int tid, int cta, int ncta, float *sh) {
  const int d4 = a.d >> 2;
  for (int r = cta; r < rows; r += ncta) {
    float *xr = a.x + (long long)r * a.d;
    float4 v[PRO_NV];
#pragma unroll
    for (int j = 0; j < PRO_NV; ++j) {
      int i = tid + j * PRO_THREADS;
      v[j] = i < d4 ? ld_f4(xr + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (a.has_in) {
      float4 gv[PRO_NV];
#pragma unroll
      for (int j = 0; j < PRO_NV; ++j) {
        int i = tid + j * PRO_THREADS;
        gv[j] = i < d4 ? gemm_val4(a.gin, r, 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int j = 0; j < PRO_NV; ++j) {
        int i = tid + j * PRO_THREADS;
        v[j].x += gv[j].x; v[j].y += gv[j].y; v[j].z += gv[j].z; v[j].w += gv[j].w;
        if (i < d4) *reinterpret_cast<float4 *>(xr + 4 * i) = v[j];
      }
    }
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < PRO_NV; ++j) ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
    float tot = pro_group_sum(ss, sh, tid);
    float inv = rsqrtf(tot / (float)a.d + a.eps);
    bool do_copy = a.copy != nullptr && (a.tap_state == nullptr || a.tap_state[a.row_seq[r]] == a.layer);
#pragma unroll
    for (int j = 0; j < PRO_NV; ++j) {
      int i = tid + j * PRO_THREADS;
      if (i >= d4) continue;
      float4 t = v[j];
      if (do_copy) *reinterpret_cast<float4 *>(a.copy + (long long)r * a.d + 4 * i) = t;
      if (a.raw) store_split4<bf16>(a.raw + r * a.lay.row_stride + 4 * i, a.lay.lo_delta, t);
      if (a.xn) {
        float4 gq = ld_f4(a.gain + 4 * i);
        store_split4<bf16>(a.xn + r * a.lay.row_stride + 4 * i, a.lay.lo_delta,
                           make_float4(t.x * inv * gq.x, t.y * inv * gq.y, t.z * inv * gq.z, t.w * inv * gq.w));
      }
    }
  }
}

__device__ __forceinline__ void pro_silu(const ProSilu &a, int rows, int tid, int cta, int ncta) {
  const int f4 = a.ff >> 2;
  const long long items = (long long)rows * f4, stride = (long long)ncta * PRO_THREADS;
  // four items per round: their loads are all in flight before the first is used
  for (long long base = (long long)cta * PRO_THREADS + tid; base < items; base += 4 * stride) {
    float4 g[4], u[4];
    int rr[4], ii[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      long long idx = base + k * stride;
      bool ok = idx < items;
      rr[k] = ok ? (int)(idx / f4) : -1;
      ii[k] = ok ? (int)(idx - (long long)rr[k] * f4) * 4 : 0;
      if (ok) { g[k] = gemm_val4(a.g, rr[k], ii[k]); u[k] = gemm_val4(a.g, rr[k], a.ff + ii[k]); }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (rr[k] < 0) continue;
      float4 o = make_float4(g[k].x / (1.f + __expf(-g[k].x)) * u[k].x, g[k].y / (1.f + __expf(-g[k].y)) * u[k].y,
                             g[k].z / (1.f + __expf(-g[k].z)) * u[k].z, g[k].w / (1.f + __expf(-g[k].w)) * u[k].w);
      store_split4<bf16>(a.act + rr[k] * a.lay.row_stride + ii[k], a.lay.lo_delta, o);
    }
  }
}

// out[r][h] = sum_c w_c O_c / sum_c w_c l_c with w_c = 2^(m_c - max m); partials are laid out
// [slot][chunk][kv head][row tile][64][hd].
__device__ __forceinline__ void pro_combine_item(const ProCombine &a, long long idx) {
  const int q4 = a.hd >> 2;
  int c4 = (int)(idx % q4);
  long long rh = idx / q4;
  int h = (int)(rh % a.H), r = (int)(rh / a.H);
  if (a.row_in && a.row_in[r] < 0) return;
  const int Hkv = a.H / a.G;
  int slot = r / a.rows_per_seq, node = r - slot * a.rows_per_seq;
  int kvh = h / a.G, rr = node * a.G + (h - kvh * a.G);
  int rt = rr >> 6, lr = rr & 63;
  const long long cstride = (long long)Hkv * a.n_rt * 64;
  const long long p0 = (((long long)slot * a.n_chunks * Hkv + kvh) * a.n_rt + rt) * 64 + lr;
  // chunks in rounds of four: (m, l) pairs and output vectors are fetched together, the running
  // maximum rescales what has been accumulated (same result as a two-pass merge up to rounding)
  float M = -INFINITY, L = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = 0; c0 < a.n_chunks; c0 += 4) {
    float2 ml[4];
    float4 o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      bool ok = c0 + k < a.n_chunks;
      long long pr = p0 + (long long)(ok ? c0 + k : c0) * cstride;
      ml[k] = ok ? __ldcg(reinterpret_cast<const float2 *>(a.part_ml + pr * 2)) : make_float2(-INFINITY, 0.f);
      o[k] = ok ? __ldcg(reinterpret_cast<const float4 *>(a.part_o + pr * a.hd + c4 * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (ml[k].x == -INFINITY) continue;
      float Mn = fmaxf(M, ml[k].x);
      float sc = exp2f(M - Mn), w = exp2f(ml[k].x - Mn);       // exp2(-inf) = 0 on the first live chunk
      L = L * sc + ml[k].y * w;
      acc.x = acc.x * sc + o[k].x * w; acc.y = acc.y * sc + o[k].y * w;
      acc.z = acc.z * sc + o[k].z * w; acc.w = acc.w * sc + o[k].w * w;
      M = Mn;
    }
  }
  float inv = L > 0.f ? 1.f / L : 0.f;
  store_split4<bf16>(a.out + r * a.lay.row_stride + h * a.hd + c4 * 4, a.lay.lo_delta,
                     make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
}
__device__ __forceinline__ void pro_combine(const ProCombine &a, int rows, int tid, int cta, int ncta) {
  const long long items = (long long)rows * a.H * (a.hd >> 2);
  for (long long idx = (long long)cta * PRO_THREADS + tid; idx < items; idx += (long long)ncta * PRO_THREADS) pro_combine_item(a, idx);
}

// tid in [0, PRO_THREADS); every prologue thread of every CTA calls this with the same arguments.
__device__ __forceinline__ void pro_run(const Prologue &p, int tid, int cta, int ncta, float *sh) {
  if (p.kind == PRO_NORM) pro_norm(p.norm, p.rows, tid, cta, ncta, sh);
  else if (p.kind == PRO_SILU) pro_silu(p.silu, p.rows, tid, cta, ncta);
  else if (p.kind == PRO_COMBINE) pro_combine(p.comb, p.rows, tid, cta, ncta);
}
