// Merge of the split-K attention partials.
//
// The attention kernels (attn_tc.cuh) cut the keys of a sequence into chunks, one CTA each; a chunk
// leaves, per query entry, the running maximum m, the sum l and the unnormalised output O of its
// keys (exp2 domain).  k_attn_combine merges them in chunk order, one thread per four output
// values, and writes the finished rows as GEMM input rows (high and low bf16 parts).
#pragma once
#include "common.cuh"
#include "rows.cuh"

#define AM_ROWS 64

// Two floats -> packed bf16 pair (high parts) and the packed pair of the remainders.
__device__ __forceinline__ void split_pair(float x, float y, uint32_t &hi, uint32_t &lo) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  float2 f = __bfloat1622float2(h);
  __nv_bfloat162 l = __floats2bfloat162_rn(x - f.x, y - f.y);
  hi = *reinterpret_cast<uint32_t *>(&h);
  lo = *reinterpret_cast<uint32_t *>(&l);
}

// What the merge kernel needs to know about the partials and the output rows.
struct AttnMergeArgs {
  const int *row_in;                // [R] or null: rows with a negative entry are idle ...
  const int *row_vis;               // ... unless this one is given and holds an entry >= 0 for the row
  int rows_per_seq, H, G;           // query rows per sequence slot, query heads, heads per KV head
  int n_chunks, n_rt;               // key chunks, 64-entry tiles per KV head
  float *part_o, *part_ml;          // [slot][chunk][kvh][rt][64][hd], [..][64][2]
  const float *part_u;              // [..][64] the chunks' u = sum p (s - m) (exp2 domain), with row_ent
  float *row_ent;                   // [R][H] entropy of each row's attention distribution, or null
  void *out;                        // [R][H*hd] rows in GEMM-input layout
  XLayout lay;
};

// Merge of the chunk partials: out[r][h] = sum_c w_c O_c / sum_c w_c l_c with w_c = 2^(m_c - max m).
// One thread per (row, head, four output columns); grid = ceil(R * H * hd / 4 / 256).  Partials are
// laid out [slot][chunk][kv head][row tile][64][hd].
template <int HD>
__global__ void __launch_bounds__(256)
k_attn_combine(AttnMergeArgs a, int R) {
  kernel_entry(TR_k_attn_combine);
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)R * a.H * (HD / 4)) return;
  constexpr int Q4 = HD >> 2;
  int c4 = (int)(idx % Q4);
  long long rh = idx / Q4;
  int h = (int)(rh % a.H), r = (int)(rh / a.H);
  if (a.row_in && a.row_in[r] < 0 && !(a.row_vis && a.row_vis[r] >= 0)) return;
  const int Hkv = a.H / a.G;
  int slot = r / a.rows_per_seq, node = r - slot * a.rows_per_seq;
  int kvh = h / a.G, rr = node * a.G + (h - kvh * a.G);
  int rt = rr >> 6, lr = rr & 63;
  const long long cstride = (long long)Hkv * a.n_rt * 64;
  const long long p0 = (((long long)slot * a.n_chunks * Hkv + kvh) * a.n_rt + rt) * 64 + lr;
  // chunks in rounds of four: (m, l) pairs and output vectors are fetched together, the running
  // maximum rescales what has been accumulated (same result as a two-pass merge up to rounding)
  float M = -INFINITY, L = 0.f, U = 0.f;
  const bool want_ent = a.row_ent != nullptr && c4 == 0;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = 0; c0 < a.n_chunks; c0 += 4) {
    float2 ml[4];
    float4 o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      bool ok = c0 + k < a.n_chunks;
      long long pr = p0 + (long long)(ok ? c0 + k : c0) * cstride;
      ml[k] = ok ? __ldcg(reinterpret_cast<const float2 *>(a.part_ml + pr * 2)) : make_float2(-INFINITY, 0.f);
      o[k] = ok ? __ldcg(reinterpret_cast<const float4 *>(a.part_o + pr * HD + c4 * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (ml[k].x == -INFINITY) continue;
      float Mn = fmaxf(M, ml[k].x);
      float sc = exp2f(M - Mn), w = exp2f(ml[k].x - Mn);       // exp2(-inf) = 0 on the first live chunk
      // u relative to the new maximum: sum p' (s - Mn) with p' = p 2^(m - Mn)
      if (want_ent) U = (L > 0.f ? sc * (U + (M - Mn) * L) : 0.f) + w * (a.part_u[p0 + (long long)(c0 + k) * cstride] + (ml[k].x - Mn) * ml[k].y);
      L = L * sc + ml[k].y * w;
      acc.x = acc.x * sc + o[k].x * w; acc.y = acc.y * sc + o[k].y * w;
      acc.z = acc.z * sc + o[k].z * w; acc.w = acc.w * sc + o[k].w * w;
      M = Mn;
    }
  }
  float inv = L > 0.f ? 1.f / L : 0.f;
  if (want_ent) a.row_ent[(long long)r * a.H + h] = L > 0.f ? logf(L) - U * 0.6931471805599453f * inv : 0.f;
  store_split4<bf16>(reinterpret_cast<bf16 *>(a.out) + r * a.lay.row_stride + h * HD + c4 * 4, a.lay.lo_delta,
                     make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
}
