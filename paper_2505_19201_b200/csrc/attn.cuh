// Attention kernels of the DREAM hot path, one warp per (query row, head):
//   - causal prefill attention with the entropy accumulators of Eq. 2 fused in,
//   - visual-token importance (column sums of the attention matrix, Section 3.3),
//   - tree-masked verification attention over the paged prefix plus the tree tail,
//   - the draft's self- and cross-attention (Eq. 1) over flat caches plus tree rows.
// Every lane holds HD/32 consecutive elements of q, k and v; a key costs one coalesced
// row load, HD/32 FMAs and a butterfly reduction.  Softmax runs online in fp32.
#pragma once
#include "common.cuh"
#include "rows.cuh"

template <int EPL, typename T> struct RowLoad;
template <int EPL> struct RowLoad<EPL, float> {
  static __device__ __forceinline__ void ld(const float *p, int lane, float (&o)[EPL]) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[e] = p[lane * EPL + e];
  }
};
template <int EPL> struct RowLoad<EPL, bf16> {
  static __device__ __forceinline__ void ld(const bf16 *p, int lane, float (&o)[EPL]) {
    const __nv_bfloat162 *p2 = reinterpret_cast<const __nv_bfloat162 *>(p + lane * EPL);
#pragma unroll
    for (int e = 0; e < EPL / 2; ++e) {
      float2 f = __bfloat1622float2(p2[e]);
      o[2 * e] = f.x; o[2 * e + 1] = f.y;
    }
  }
};

// Lane's share of the query of (row, head) rh; bf16 configurations store a high and a low row.
template <int EPL, typename T> struct QLoad;
template <int EPL> struct QLoad<EPL, float> {
  static __device__ __forceinline__ void ld(const void *qbuf, long long rh, int lane, float (&o)[EPL]) {
    RowLoad<EPL, float>::ld((const float *)qbuf + rh * (EPL * 32), lane, o);
  }
};
template <int EPL> struct QLoad<EPL, bf16> {
  static __device__ __forceinline__ void ld(const void *qbuf, long long rh, int lane, float (&o)[EPL]) {
    float lo[EPL];
    RowLoad<EPL, bf16>::ld((const bf16 *)qbuf + rh * 2 * (EPL * 32), lane, o);
    RowLoad<EPL, bf16>::ld((const bf16 *)qbuf + rh * 2 * (EPL * 32) + EPL * 32, lane, lo);
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[e] += lo[e];
  }
};

// Online-softmax state of one (row, head): running max m, Z = sum e^{s-m}, the weighted
// value sum, and U = sum e^{s-m}(s-m) for the entropy  H = ln Z - U/Z  (Eq. 2, inner sum).
template <int EPL> struct Soft {
  float m, z, u, acc[EPL];
  __device__ __forceinline__ void init() {
    m = -INFINITY; z = 0.f; u = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  }
  template <bool ENT>
  __device__ __forceinline__ void push(float s, const float (&v)[EPL]) {
    if (s > m) {
      float delta = s - m;                    // may be +inf on the first key
      float sc = __expf(-delta);              // 0 when m was -inf
      if (ENT) u = z > 0.f ? sc * (u - delta * z) : 0.f;
      z *= sc;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] *= sc;
      m = s;
    }
    float p = __expf(s - m);
    z += p;
    if (ENT) u += p * (s - m);
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += p * v[e];
  }
};

template <int EPL>
__device__ __forceinline__ float dot_lane(const float (&a)[EPL], const float (&b)[EPL]) {
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < EPL; ++e) s += a[e] * b[e];
  return warp_sum(s);
}

#define ATT_WARPS 8

// ---------------------------------------------------------------------------------------
// Causal self-attention of the n prompt rows at one layer.  A warp owns ATT_PF_ROWS consecutive
// rows of one head, so a key/value row fetched from the cache serves all of them; two keys are
// in flight at a time (their loads and butterfly reductions overlap) and each row's softmax state
// takes its keys one by one in ascending order.  grid (ceil(n / (8 * ATT_PF_ROWS)), H).
// Outputs: attn_out, rows of H*hd values (element type, input of the O projection) in chunks of
// chunk_rows rows, chunk_stride elements apart, each laid out as `lay` says; lse [H][n] (row
// log-sum-exp of the scaled scores, for the importance pass), ent [H][n] row entropies.
#define ATT_PF_ROWS 4
template <typename T, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32)
k_attn_prefill(const void *__restrict__ qbuf, PagedKV kv, int seq, int n, int H, float scale,
               T *attn_out, XLayout lay, int chunk_rows, long long chunk_stride, float *lse, float *ent) {
  constexpr int EPL = HD / 32, RW = ATT_PF_ROWS;
  kernel_entry(TR_k_attn_prefill);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int i0 = (blockIdx.x * ATT_WARPS + w) * RW, h = blockIdx.y;
  if (i0 >= n) return;
  const int nr = min(RW, n - i0);
  int kvh = h / (H / kv.hkv);
  const T *Kp = (const T *)kv.base, *Vp = (const T *)kv.base + kv.kv_stride;
  float q[RW][EPL];
  Soft<EPL> st[RW];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    QLoad<EPL, T>::ld(qbuf, (long long)min(i0 + r, n - 1) * H + h, lane, q[r]);
#pragma unroll
    for (int e = 0; e < EPL; ++e) q[r][e] *= scale;
    st[r].init();
  }
  const int jmax = i0 + nr - 1;
  for (int j = 0; j <= jmax; j += 2) {
    float k0[EPL], v0[EPL], k1[EPL], v1[EPL], s0[RW], s1[RW];
    const bool two = j + 1 <= jmax;
    long long o0 = kv.off(seq, j, kvh), o1 = kv.off(seq, two ? j + 1 : j, kvh);
    RowLoad<EPL, T>::ld(Kp + o0, lane, k0);
    RowLoad<EPL, T>::ld(Vp + o0, lane, v0);
    RowLoad<EPL, T>::ld(Kp + o1, lane, k1);
    RowLoad<EPL, T>::ld(Vp + o1, lane, v1);
#pragma unroll
    for (int r = 0; r < RW; ++r) { s0[r] = dot_lane<EPL>(q[r], k0); s1[r] = dot_lane<EPL>(q[r], k1); }
#pragma unroll
    for (int r = 0; r < RW; ++r) {
      if (r < nr && j <= i0 + r) st[r].template push<true>(s0[r], v0);
      if (r < nr && two && j + 1 <= i0 + r) st[r].template push<true>(s1[r], v1);
    }
  }
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    if (r >= nr) break;
    const int i = i0 + r;
    float inv = 1.f / st[r].z;
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      store_split<T>(attn_out + (i / chunk_rows) * chunk_stride + (i % chunk_rows) * lay.row_stride + h * HD + lane * EPL + e,
                     lay.lo_delta, st[r].acc[e] * inv);
    if (lane == 0) {
      lse[(long long)h * n + i] = st[r].m + logf(st[r].z);
      ent[(long long)h * n + i] = logf(st[r].z) - st[r].u / st[r].z;
    }
  }
}

// AE(l) = mean over rows and heads of the row entropies (Eq. 2).  One block, fixed order.
// sum_out (may be null) receives the sum itself: the start of the running form of Eq. 2.
__global__ void k_entropy_mean(const float *__restrict__ ent, int count, float *out, float *sum_out) {
  __shared__ float sh[33];
  kernel_entry(TR_k_entropy_mean);
  float s = 0.f;
  for (int i = threadIdx.x; i < count; i += blockDim.x) s += ent[i];
  float t = block_sum(s, sh);
  if (threadIdx.x == 0) { *out = t / (float)count; if (sum_out) *sum_out = t; }
}


// Importance of visual token j at this layer (Section 3.3): the attention weight it receives,
// summed over the later query rows (and its own row when include_self) and over heads.
// One warp per (visual column, head), grid (ceil(v / 8), H): rows ascending, four in flight at a
// time, added in row order; k_colsum_heads then adds the heads in ascending order: a fixed order.
template <typename T, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32)
k_colsum(const void *__restrict__ qbuf, PagedKV kv, int seq, int n, int H, float scale,
         const float *__restrict__ lse, int vis_start, int v, int include_self, float *part /* [H][v] */) {
  constexpr int EPL = HD / 32;
  kernel_entry(TR_k_colsum);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int jv = blockIdx.x * ATT_WARPS + w, h = blockIdx.y;
  if (jv >= v) return;
  int j = vis_start + jv;
  int kvh = h / (H / kv.hkv);
  float k[EPL];
  RowLoad<EPL, T>::ld((const T *)kv.base + kv.off(seq, j, kvh), lane, k);
  const float *lse_h = lse + (long long)h * n;
  float hs = 0.f;
  int i = include_self ? j : j + 1;
  for (; i + 3 < n; i += 4) {
    float q0[EPL], q1[EPL], q2[EPL], q3[EPL];
    QLoad<EPL, T>::ld(qbuf, (long long)i * H + h, lane, q0);
    QLoad<EPL, T>::ld(qbuf, (long long)(i + 1) * H + h, lane, q1);
    QLoad<EPL, T>::ld(qbuf, (long long)(i + 2) * H + h, lane, q2);
    QLoad<EPL, T>::ld(qbuf, (long long)(i + 3) * H + h, lane, q3);
    float l0 = lse_h[i], l1 = lse_h[i + 1], l2 = lse_h[i + 2], l3 = lse_h[i + 3];
    float s0 = dot_lane<EPL>(q0, k), s1 = dot_lane<EPL>(q1, k), s2 = dot_lane<EPL>(q2, k), s3 = dot_lane<EPL>(q3, k);
    hs += __expf(s0 * scale - l0);
    hs += __expf(s1 * scale - l1);
    hs += __expf(s2 * scale - l2);
    hs += __expf(s3 * scale - l3);
  }
  for (; i < n; ++i) {
    float q[EPL];
    QLoad<EPL, T>::ld(qbuf, (long long)i * H + h, lane, q);
    hs += __expf(dot_lane<EPL>(q, k) * scale - lse_h[i]);
  }
  if (lane == 0) part[(long long)h * v + jv] = hs;
}

// score[jv] = sum over heads, ascending, of the per-head column sums.
__global__ void k_colsum_heads(const float *__restrict__ part, int H, int v, float *score) {
  kernel_entry(TR_k_colsum);
  int jv = blockIdx.x * blockDim.x + threadIdx.x;
  if (jv >= v) return;
  float tot = 0.f;
  for (int h = 0; h < H; ++h) tot += part[(long long)h * v + jv];
  score[jv] = tot;
}

// ---------------------------------------------------------------------------------------
// Tree-masked verification attention (Section 3.1).  Row r = tree node of sequence
// row_seq[r]; it sees prefix slots [0, P) and tail slots P + j for every j in its
// ancestor-or-self bit set.  grid (ceil(R/8), H).
// row_ent (ENT only): [R][H] entropy of the row's attention distribution.
template <typename T, int HD, bool ENT>
__global__ void __launch_bounds__(ATT_WARPS * 32)
k_attn_tree(const void *__restrict__ qbuf, PagedKV kv, const int *__restrict__ row_seq,
            const int *__restrict__ row_node, const int *__restrict__ P_state,
            const uint32_t *__restrict__ mask, int R, int T_nodes, int H, float scale, T *attn_out,
            XLayout lay, float *row_ent) {
  constexpr int EPL = HD / 32;
  kernel_entry(TR_k_attn_tree);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int r = blockIdx.x * ATT_WARPS + w, h = blockIdx.y;
  if (r >= R) return;
  int seq = row_seq[r], P = P_state[seq];
  int kvh = h / (H / kv.hkv);
  const T *Kp = (const T *)kv.base, *Vp = (const T *)kv.base + kv.kv_stride;
  float q[EPL], k[EPL], v[EPL];
  QLoad<EPL, T>::ld(qbuf, (long long)r * H + h, lane, q);
#pragma unroll
  for (int e = 0; e < EPL; ++e) q[e] *= scale;
  Soft<EPL> st;
  st.init();
  for (int j = 0; j < P; ++j) {
    long long o = kv.off(seq, j, kvh);
    RowLoad<EPL, T>::ld(Kp + o, lane, k);
    RowLoad<EPL, T>::ld(Vp + o, lane, v);
    st.template push<ENT>(dot_lane<EPL>(q, k), v);
  }
  const uint32_t *mr = mask + (long long)r * 4;
  for (int j = 0; j < T_nodes; ++j) {
    if (!((mr[j >> 5] >> (j & 31)) & 1u)) continue;
    long long o = kv.off(seq, P + j, kvh);
    RowLoad<EPL, T>::ld(Kp + o, lane, k);
    RowLoad<EPL, T>::ld(Vp + o, lane, v);
    st.template push<ENT>(dot_lane<EPL>(q, k), v);
  }
  (void)row_node;
  float inv = 1.f / st.z;
  if (ENT && lane == 0) row_ent[(long long)r * H + h] = logf(st.z) - st.u * inv;
#pragma unroll
  for (int e = 0; e < EPL; ++e)
    store_split<T>(attn_out + r * lay.row_stride + h * HD + lane * EPL + e, lay.lo_delta, st.acc[e] * inv);
}

// ---------------------------------------------------------------------------------------
// Draft attention over a flat cache: permanent rows [0, nperm[seq]) are all visible, then
// tree-region rows nperm + j for each j in the row's ancestor set (self excluded when
// strict: cross-attention reads the draft features of strict ancestors only, Section 3.1).
// Rows with row_in < 0 are idle, unless row_vis is given and holds v >= 0 for the row: such a row
// sees the rows [0, v) and nothing else (none at all when v = 0: its output is zero).  grid (ceil(R/8), H).
template <typename T, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32)
k_attn_draft(const void *__restrict__ qbuf, FlatKV kv, const int *__restrict__ row_seq,
             const int *__restrict__ row_in, const int *__restrict__ row_vis, const int *__restrict__ nperm,
             const unsigned long long *__restrict__ anc, int anc_stride, int strict, int R, int H,
             float scale, T *attn_out, XLayout lay) {
  constexpr int EPL = HD / 32;
  kernel_entry(TR_k_attn_draft);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int r = blockIdx.x * ATT_WARPS + w, h = blockIdx.y;
  if (r >= R) return;
  int in = row_in ? row_in[r] : 0;
  const int rv = row_vis ? row_vis[r] : -1;
  if (in < 0 && rv < 0) return;
  int seq = row_seq[r], np = rv >= 0 ? rv : nperm[seq];
  int kvh = h / (H / kv.hkv);
  const float *base = (const float *)kv.base;          // fp32 configurations only
  long long ok = kv.off(seq, 0, kvh, 0), ov = kv.off(seq, 1, kvh, 0);
  float q[EPL], k[EPL], v[EPL];
  QLoad<EPL, T>::ld(qbuf, (long long)r * H + h, lane, q);
#pragma unroll
  for (int e = 0; e < EPL; ++e) q[e] *= scale;
  Soft<EPL> st;
  st.init();
  for (int j = 0; j < np; ++j) {
    RowLoad<EPL, float>::ld(base + ok + (long long)j * HD, lane, k);
    RowLoad<EPL, float>::ld(base + ov + (long long)j * HD, lane, v);
    st.template push<false>(dot_lane<EPL>(q, k), v);
  }
  unsigned long long bits = rv >= 0 ? 0ull : anc[(long long)seq * anc_stride + in];
  if (strict && rv < 0) bits &= ~(1ull << in);
  while (bits) {
    int j = __ffsll((long long)bits) - 1;
    bits &= bits - 1;
    RowLoad<EPL, float>::ld(base + ok + (long long)(np + j) * HD, lane, k);
    RowLoad<EPL, float>::ld(base + ov + (long long)(np + j) * HD, lane, v);
    st.template push<false>(dot_lane<EPL>(q, k), v);
  }
  float inv = st.z > 0.f ? 1.f / st.z : 0.f;
#pragma unroll
  for (int e = 0; e < EPL; ++e)
    store_split<T>(attn_out + r * lay.row_stride + h * HD + lane * EPL + e, lay.lo_delta, st.acc[e] * inv);
}
