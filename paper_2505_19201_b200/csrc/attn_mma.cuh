// Split-K decode attention on the warp-level tensor-core path (mma.sync m16n8k16, bf16 inputs,
// fp32 accumulate) for the few-query, many-key attention of the loop: tree-masked verification
// over the paged target cache (Section 3.1) and the draft's self- and cross-attention over its
// flat caches (Eq. 1).
//
// A CTA owns 64 query rows (row = (tree node, query head of one KV-head group)), one KV head and
// one chunk of keys.  It walks the chunk in blocks of AM_KBLK keys staged in shared memory by
// cp.async (double buffered, 16-byte segments, padded rows: conflict-free ldmatrix), computes
// S = Q K^T, an online softmax in the exp2 domain, and O += P V, all in registers.  Queries and
// probabilities enter the tensor cores as a high and a low bf16 part, so the products keep ~16
// mantissa bits; K and V are used as stored.  Each chunk leaves (m, l, O) partials that
// k_attn_combine merges in chunk order, one thread per four output values, and writes as GEMM
// input rows (a single chunk writes them itself).  Visible keys of a row: every key below
// prefix_len[seq], plus tail key j for every bit j of the row's mask.
#pragma once
#include "common.cuh"
#include "rows.cuh"

#define AM_ROWS 64
#define AM_THREADS 128

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Two floats -> packed bf16 pair (high parts) and the packed pair of the remainders.
__device__ __forceinline__ void split_pair(float x, float y, uint32_t &hi, uint32_t &lo) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  float2 f = __bfloat1622float2(h);
  __nv_bfloat162 l = __floats2bfloat162_rn(x - f.x, y - f.y);
  hi = *reinterpret_cast<uint32_t *>(&h);
  lo = *reinterpret_cast<uint32_t *>(&l);
}

// Flat draft cache in bf16 with a high and a low row per key: [seq][2][H_kv][cap][2][hd].
struct FlatKV2 {
  bf16 *base;
  int cap, hkv, hd;
  __device__ __forceinline__ long long off(int seq, int kv, int kvh, int row) const {
    return (((((long long)seq * 2 + kv) * hkv + kvh) * cap + row) * 2) * hd;
  }
};

struct AttnMmaArgs {
  const bf16 *q;                    // [R][H][2][hd] queries (rotary applied, unscaled): high row, low row
  int slot_seq[DREAM_MAX_BATCH];    // sequence of each query-row slot (grid z)
  const int *row_in;                // [R] or null: rows with a negative entry are idle; index into anc
  const int *prefix_len;            // by sequence: keys [0, prefix) are visible to every row
  const uint32_t *mask;             // [R][4] visible tail keys, or null when anc is given
  const unsigned long long *anc;    // [seq][anc_stride] ancestor-or-self bits over tail keys, or null
  int anc_stride, strict;           // strict: a row does not see its own tail key
  int rows_per_seq, tail_len, H, G; // query rows per sequence slot, tail keys, query heads, heads per KV head
  float scale_log2;                 // softmax scale times log2(e)
  int n_chunks, blocks_per_chunk, n_rt;
  float *part_o, *part_ml;          // [slot][chunk][kvh][rt][64][hd], [..][64][2]
  void *out;                        // [R][H*hd] rows in GEMM-input layout
  XLayout lay;
  L2Prefetch next_w;                // weights of the GEMM that follows, pulled into L2 meanwhile
  PagedKV paged;                    // PAGED kernels
  FlatKV2 flat;                     // flat kernels
};

template <int HD> struct AmShape {
  static constexpr int KBLK = HD == 256 ? 32 : 64;     // keys per shared-memory block
  static constexpr int LD = HD + 8;                    // padded row, elements
};

// Shared memory: Qh, Ql [64][LD]; then per buffer (x2): K (and K_lo), V (and V_lo) [KBLK][LD].
template <int HD, bool PAGED>
constexpr size_t attn_mma_smem() {
  return (size_t)2 * AM_ROWS * AmShape<HD>::LD * 2 + (size_t)2 * (PAGED ? 2 : 4) * AmShape<HD>::KBLK * AmShape<HD>::LD * 2 + AM_ROWS * 24;
}

// One block of KBLK keys for the sixteen query rows of a warp: S = Q K^T (queries as high + low
// parts; K as stored, plus its low plane when PLANES == 2), tail mask, online softmax in the exp2
// domain, O += P V (probabilities as high + low parts).  Kb / Vb: the block's K and V planes in
// shared memory; mw0 / mw1: visible-tail-key bits of the thread's two rows.
template <int HD, int PLANES>
__device__ __forceinline__ void attn_block(const bf16 *Kb, const bf16 *Vb, uint32_t qh_addr, uint32_t ql_addr, int k_row, int k_col,
                                           int v_row, int v_col, int t, int j0, int P, int tail_len, float scale_log2,
                                           const uint32_t (&mw0)[4], const uint32_t (&mw1)[4],
                                           float (&o_acc)[HD / 8][4], float (&m_run)[2], float (&l_run)[2]) {
  constexpr int KBLK = AmShape<HD>::KBLK, LD = AmShape<HD>::LD;
  constexpr int NT_S = KBLK / 8, NT_O = HD / 8, PLANE_ELEMS = KBLK * LD;
  constexpr bool PAGED = PLANES == 1;
  // ---- S = Q K^T
  float s[NT_S][4];
#pragma unroll
  for (int n = 0; n < NT_S; ++n) { s[n][0] = 0.f; s[n][1] = 0.f; s[n][2] = 0.f; s[n][3] = 0.f; }
#pragma unroll
  for (int ks = 0; ks < HD / 16; ++ks) {
    uint32_t ah0, ah1, ah2, ah3, al0, al1, al2, al3;
    ldsm_x4(qh_addr + ks * 32, ah0, ah1, ah2, ah3);
    ldsm_x4(ql_addr + ks * 32, al0, al1, al2, al3);
#pragma unroll
    for (int np = 0; np < NT_S / 2; ++np) {
      uint32_t kb0, kb1, kb2, kb3;
      uint32_t ka = smem_addr(Kb + (np * 16 + k_row) * LD + ks * 16 + k_col);
      ldsm_x4(ka, kb0, kb1, kb2, kb3);
      mma_16816(s[2 * np], ah0, ah1, ah2, ah3, kb0, kb1);
      mma_16816(s[2 * np], al0, al1, al2, al3, kb0, kb1);
      mma_16816(s[2 * np + 1], ah0, ah1, ah2, ah3, kb2, kb3);
      mma_16816(s[2 * np + 1], al0, al1, al2, al3, kb2, kb3);
      if (!PAGED) {
        ldsm_x4(ka + PLANE_ELEMS * 2, kb0, kb1, kb2, kb3);
        mma_16816(s[2 * np], ah0, ah1, ah2, ah3, kb0, kb1);
        mma_16816(s[2 * np + 1], ah0, ah1, ah2, ah3, kb2, kb3);
      }
    }
  }
  // ---- scale, mask, online softmax (exp2 domain)
  const bool need_mask = j0 + KBLK > P;
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int n = 0; n < NT_S; ++n) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float v = s[n][e] * scale_log2;
      if (need_mask) {
        int j = j0 + n * 8 + 2 * t + (e & 1);
        bool vis = j < P;
        if (!vis) {
          int jt = j - P;
          if (jt < tail_len) {
            uint32_t wsel = (e >> 1) ? ((jt >> 5) == 0 ? mw1[0] : (jt >> 5) == 1 ? mw1[1] : (jt >> 5) == 2 ? mw1[2] : mw1[3])
                                     : ((jt >> 5) == 0 ? mw0[0] : (jt >> 5) == 1 ? mw0[1] : (jt >> 5) == 2 ? mw0[2] : mw0[3]);
            vis = (wsel >> (jt & 31)) & 1u;
          }
        }
        if (!vis) v = -INFINITY;
      }
      s[n][e] = v;
      if (e >> 1) mx1 = fmaxf(mx1, v); else mx0 = fmaxf(mx0, v);
    }
  }
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
  float base0 = mn0 == -INFINITY ? 0.f : mn0, base1 = mn1 == -INFINITY ? 0.f : mn1;
  float corr0 = exp2f(m_run[0] - base0), corr1 = exp2f(m_run[1] - base1);
  m_run[0] = mn0; m_run[1] = mn1;
  l_run[0] *= corr0; l_run[1] *= corr1;
#pragma unroll
  for (int n = 0; n < NT_O; ++n) { o_acc[n][0] *= corr0; o_acc[n][1] *= corr0; o_acc[n][2] *= corr1; o_acc[n][3] *= corr1; }
#pragma unroll
  for (int n = 0; n < NT_S; ++n) {
    s[n][0] = exp2f(s[n][0] - base0); s[n][1] = exp2f(s[n][1] - base0);
    s[n][2] = exp2f(s[n][2] - base1); s[n][3] = exp2f(s[n][3] - base1);
    l_run[0] += s[n][0] + s[n][1]; l_run[1] += s[n][2] + s[n][3];
  }
  // ---- O += P V
#pragma unroll
  for (int kk = 0; kk < KBLK / 16; ++kk) {
    uint32_t ph0, ph1, ph2, ph3, pl0, pl1, pl2, pl3;
    split_pair(s[2 * kk][0], s[2 * kk][1], ph0, pl0);
    split_pair(s[2 * kk][2], s[2 * kk][3], ph1, pl1);
    split_pair(s[2 * kk + 1][0], s[2 * kk + 1][1], ph2, pl2);
    split_pair(s[2 * kk + 1][2], s[2 * kk + 1][3], ph3, pl3);
#pragma unroll
    for (int nd = 0; nd < HD / 16; ++nd) {
      uint32_t vb0, vb1, vb2, vb3;
      uint32_t va = smem_addr(Vb + (kk * 16 + v_row) * LD + nd * 16 + v_col);
      ldsm_x4_t(va, vb0, vb1, vb2, vb3);
      mma_16816(o_acc[2 * nd], ph0, ph1, ph2, ph3, vb0, vb1);
      mma_16816(o_acc[2 * nd], pl0, pl1, pl2, pl3, vb0, vb1);
      mma_16816(o_acc[2 * nd + 1], ph0, ph1, ph2, ph3, vb2, vb3);
      mma_16816(o_acc[2 * nd + 1], pl0, pl1, pl2, pl3, vb2, vb3);
      if (!PAGED) {
        ldsm_x4_t(va + PLANE_ELEMS * 2, vb0, vb1, vb2, vb3);
        mma_16816(o_acc[2 * nd], ph0, ph1, ph2, ph3, vb0, vb1);
        mma_16816(o_acc[2 * nd + 1], ph0, ph1, ph2, ph3, vb2, vb3);
      }
    }
  }
}

template <int HD, bool PAGED>
__global__ void __launch_bounds__(AM_THREADS)
k_attn_mma(AttnMmaArgs a) {
  constexpr int KBLK = AmShape<HD>::KBLK, LD = AmShape<HD>::LD;
  constexpr int NT_S = KBLK / 8, NT_O = HD / 8, PLANES = PAGED ? 1 : 2;
  constexpr int PLANE_ELEMS = KBLK * LD, BUF_ELEMS = 2 * PLANES * PLANE_ELEMS;   // K planes then V planes
  extern __shared__ __align__(16) uint8_t am_smem[];
  bf16 *Qh = reinterpret_cast<bf16 *>(am_smem), *Ql = Qh + AM_ROWS * LD, *KV = Ql + AM_ROWS * LD;
  uint32_t *mwords = reinterpret_cast<uint32_t *>(KV + 2 * BUF_ELEMS);          // [64][4]
  int *row_r = reinterpret_cast<int *>(mwords + AM_ROWS * 4), *row_h = row_r + AM_ROWS;
  l2_prefetch_slice(a.next_w, blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z), gridDim.x * gridDim.y * gridDim.z);
  kernel_entry_late(TR_k_attn_mma);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int chunk = blockIdx.x, kvh = blockIdx.y / a.n_rt, rt = blockIdx.y - kvh * a.n_rt, slot = blockIdx.z;
  const int Hkv = a.H / a.G;
  const int r_base = slot * a.rows_per_seq;
  const int seq = a.slot_seq[slot];
  if (PAGED && tid < a.blocks_per_chunk + 1) {       // page-table entries of this chunk's blocks, on their way to L1 meanwhile
    const int j = min((chunk * a.blocks_per_chunk + tid) * KBLK, a.paged.pages_per_seq * a.paged.page_tokens - 1);
    asm volatile("prefetch.global.L1 [%0];" ::"l"(a.paged.page_table + seq * a.paged.pages_per_seq + (j >> a.paged.page_shift)));
  }
  const int P = a.prefix_len[seq];
  const int total_keys = P + a.tail_len;
  const int nb = (total_keys + KBLK - 1) / KBLK;
  const int b0 = chunk * a.blocks_per_chunk, b1 = min(nb, b0 + a.blocks_per_chunk);
  const int rows_total = a.rows_per_seq * a.G;

  auto load_block = [&](int blk, int buf, bool commit) {
    bf16 *dstb = KV + buf * BUF_ELEMS;
    for (int idx = tid; idx < KBLK * (HD / 8); idx += AM_THREADS) {
      int row = idx / (HD / 8), sg = idx - row * (HD / 8);
      int j = blk * KBLK + row;
      bool ok = j < total_keys;
      uint32_t dk = smem_addr(dstb + row * LD + sg * 8), dv = dk + PLANES * PLANE_ELEMS * 2;
      if (PAGED) {
        const bf16 *Kp = (const bf16 *)a.paged.base, *Vp = Kp + a.paged.kv_stride;
        long long o = ok ? a.paged.off(seq, j, kvh) + sg * 8 : 0;
        cp_async16(dk, Kp + o, ok ? 16 : 0);
        cp_async16(dv, Vp + o, ok ? 16 : 0);
      } else {
        long long ok_ = ok ? a.flat.off(seq, 0, kvh, j) + sg * 8 : 0, ov_ = ok ? a.flat.off(seq, 1, kvh, j) + sg * 8 : 0;
        cp_async16(dk, a.flat.base + ok_, ok ? 16 : 0);
        cp_async16(dk + PLANE_ELEMS * 2, a.flat.base + ok_ + (ok ? HD : 0), ok ? 16 : 0);
        cp_async16(dv, a.flat.base + ov_, ok ? 16 : 0);
        cp_async16(dv + PLANE_ELEMS * 2, a.flat.base + ov_ + (ok ? HD : 0), ok ? 16 : 0);
      }
    }
    if (commit) cp_async_commit();
  };

  // the first K/V block does not depend on the row table: its copies start before the table is built
  if (b0 < b1) load_block(b0, 0, false);
  // ---- row table: global row, head and tail mask of each of the 64 rows
  if (tid < AM_ROWS) {
    int rr = rt * AM_ROWS + tid, r = -1, h = 0;
    uint32_t mw[4] = {0u, 0u, 0u, 0u};
    if (rr < rows_total) {
      int node = rr / a.G;
      r = r_base + node; h = kvh * a.G + (rr - node * a.G);
      int in = a.row_in ? a.row_in[r] : 0;
      if (in < 0) r = -1;
      else if (a.anc) {
        unsigned long long bits = a.anc[(long long)seq * a.anc_stride + in];
        if (a.strict) bits &= ~(1ull << in);
        mw[0] = (uint32_t)bits; mw[1] = (uint32_t)(bits >> 32);
      } else {
        for (int wd = 0; wd < 4; ++wd) mw[wd] = a.mask[(long long)r * 4 + wd];
      }
    }
    row_r[tid] = r; row_h[tid] = h;
    for (int wd = 0; wd < 4; ++wd) mwords[tid * 4 + wd] = mw[wd];
  }
  __syncthreads();
  // ---- queries: high and low rows copied asynchronously (same group as the first K/V block)
  for (int idx = tid; idx < AM_ROWS * (HD / 8); idx += AM_THREADS) {
    int lr = idx / (HD / 8), sg = idx - lr * (HD / 8);
    int r = row_r[lr];
    const bf16 *src = a.q + (r >= 0 ? ((long long)r * a.H + row_h[lr]) * 2 * HD + sg * 8 : 0);
    cp_async16(smem_addr(Qh + lr * LD + sg * 8), src, r >= 0 ? 16 : 0);
    cp_async16(smem_addr(Ql + lr * LD + sg * 8), src + (r >= 0 ? HD : 0), r >= 0 ? 16 : 0);
  }

  cp_async_commit();

  float o_acc[NT_O][4];
#pragma unroll
  for (int n = 0; n < NT_O; ++n) { o_acc[n][0] = 0.f; o_acc[n][1] = 0.f; o_acc[n][2] = 0.f; o_acc[n][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  uint32_t mw0[4], mw1[4];
#pragma unroll
  for (int wd = 0; wd < 4; ++wd) { mw0[wd] = mwords[(warp * 16 + g) * 4 + wd]; mw1[wd] = mwords[(warp * 16 + g + 8) * 4 + wd]; }

  // a warp whose sixteen rows are all idle (few query rows: the draft's passes) only keeps the
  // copies and barriers going
  const bool warp_live = __any_sync(0xffffffffu, row_r[warp * 16 + (lane & 15)] >= 0);

  const int mi = lane >> 3, l7 = lane & 7;
  const uint32_t qh_addr = smem_addr(Qh + (warp * 16 + l7 + (mi & 1) * 8) * LD + (mi >> 1) * 8);
  const uint32_t ql_addr = qh_addr + AM_ROWS * LD * 2;
  const int k_row = l7 + (mi >> 1) * 8, k_col = (mi & 1) * 8;          // K fragments (non-transposed)
  const int v_row = l7 + (mi & 1) * 8, v_col = (mi >> 1) * 8;          // V fragments (transposed)

  if (b0 >= b1) cp_async_wait<0>();
  for (int blk = b0; blk < b1; ++blk) {
    const int buf = (blk - b0) & 1;
    if (blk + 1 < b1) { load_block(blk + 1, buf ^ 1, true); cp_async_wait<1>(); } else cp_async_wait<0>();
    __syncthreads();
    const bf16 *Kb = KV + buf * BUF_ELEMS, *Vb = Kb + PLANES * PLANE_ELEMS;
    if (!warp_live) { __syncthreads(); continue; }
    attn_block<HD, PLANES>(Kb, Vb, qh_addr, ql_addr, k_row, k_col, v_row, v_col, t, blk * KBLK, P, a.tail_len, a.scale_log2,
                           mw0, mw1, o_acc, m_run, l_run);
    __syncthreads();
  }
  pdl_trigger();                    // the keys are done: the GEMM kernel that follows may take the SMs
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1); l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1); l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);

  if (!warp_live) return;
  bf16 *out = reinterpret_cast<bf16 *>(a.out);
  if (a.n_chunks == 1) {
#pragma unroll
    for (int rs = 0; rs < 2; ++rs) {
      int lr = warp * 16 + g + rs * 8, r = row_r[lr];
      if (r < 0) continue;
      float inv = l_run[rs] > 0.f ? 1.f / l_run[rs] : 0.f;
      bf16 *dst = out + r * a.lay.row_stride + row_h[lr] * HD + 2 * t;
#pragma unroll
      for (int n = 0; n < NT_O; ++n) {
        uint32_t hi, lo;
        split_pair(o_acc[n][rs * 2] * inv, o_acc[n][rs * 2 + 1] * inv, hi, lo);
        *reinterpret_cast<uint32_t *>(dst + n * 8) = hi;
        if (a.lay.lo_delta) *reinterpret_cast<uint32_t *>(dst + n * 8 + a.lay.lo_delta) = lo;
      }
    }
    return;
  }
  // ---- partials of this chunk
  const long long pbase = ((((long long)slot * a.n_chunks + chunk) * Hkv + kvh) * a.n_rt + rt) * AM_ROWS;
#pragma unroll
  for (int rs = 0; rs < 2; ++rs) {
    int lr = warp * 16 + g + rs * 8;
    float *po = a.part_o + (pbase + lr) * HD + 2 * t;
#pragma unroll
    for (int n = 0; n < NT_O; ++n) *reinterpret_cast<float2 *>(po + n * 8) = make_float2(o_acc[n][rs * 2], o_acc[n][rs * 2 + 1]);
    if (t == 0) *reinterpret_cast<float2 *>(a.part_ml + (pbase + lr) * 2) = make_float2(m_run[rs], l_run[rs]);
  }
}

// Merge of the chunk partials: out[r][h] = sum_c w_c O_c / sum_c w_c l_c with w_c = 2^(m_c - max m).
// One thread per (row, head, four output columns); grid = ceil(R * H * hd / 4 / 256).  Partials are
// laid out [slot][chunk][kv head][row tile][64][hd].
template <int HD>
__global__ void __launch_bounds__(256)
k_attn_combine(AttnMmaArgs a, int R) {
  kernel_entry(TR_k_attn_combine);
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)R * a.H * (HD / 4)) return;
  constexpr int Q4 = HD >> 2;
  int c4 = (int)(idx % Q4);
  long long rh = idx / Q4;
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
      o[k] = ok ? __ldcg(reinterpret_cast<const float4 *>(a.part_o + pr * HD + c4 * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
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
  store_split4<bf16>(reinterpret_cast<bf16 *>(a.out) + r * a.lay.row_stride + h * HD + c4 * 4, a.lay.lo_delta,
                     make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
}
