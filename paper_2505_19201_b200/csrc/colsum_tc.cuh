// Visual-token importance on the tcgen05 tensor cores (Section 3.3): the attention weight a visual
// token receives at one layer, summed over the later query rows, per head.
//
// The prefill attention has left every row's log-sum-exp, so a weight is exp(s_ij - lse_i) and the
// column sums need the scores once more, nothing else.  Here the KEYS sit on the MMA's M side: a CTA
// owns 128 consecutive key positions of one query head and keeps their K rows in shared memory as
// the A operand; the query rows stream past as the B operand, NQ at a time (their high and their
// low bf16 part: two MMA chains into one accumulator), so that S^T = K Q^T lands in TMEM with one
// key per lane.  Each softmax thread then owns one column of the attention matrix and adds up
// exp2(s * scale - lse) over the rows that may see it, in registers: no reduction across threads.
// Warp roles: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..5 = one key per thread.  Two
// accumulators and two query stages alternate.  Every mbarrier wait is bounded; on expiry the
// kernel raises the status word and leaves.
#pragma once
#include "attn_tc.cuh"

#define CS_THREADS 192
#define CS_KEYS 128

template <int HD> struct CsShape {
  static constexpr int KP = HD / 64;                       // 64-column panels per row
  static constexpr int NQ = HD == 256 ? 64 : 128;          // query rows per step
  static constexpr int K_BYTES = KP * CS_KEYS * 128;       // the key tile
  static constexpr int Q_STAGE = 2 * KP * NQ * 128;        // high and low plane of NQ query rows
  static constexpr size_t SMEM = 1024 + K_BYTES + 2 * Q_STAGE + 256;
};

struct ColsumTcArgs {
  int seq, n, H, G;                 // sequence, prompt rows, query heads, heads per KV head
  int vis_start, v, include_self;   // the visual span; 1: a token's attention to itself counts
  int key0;                         // first key of tile 0 (vis_start rounded down to a multiple of 64)
  float scale_log2;
  const float *lse;                 // [H][n] natural-log log-sum-exp of every row
  float *part;                      // [H][v] per-head sums
  const int *page_table;
  int pages_per_seq, page_tokens, page_shift, hkv;
  int *status;
};

template <int HD>
__global__ void __launch_bounds__(CS_THREADS, 1)
k_colsum_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ ColsumTcArgs a) {
  using Sh = CsShape<HD>;
  constexpr int KP = Sh::KP, NQ = Sh::NQ;
  extern __shared__ uint8_t cs_smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)cs_smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *k_s = smem, *q_s = k_s + Sh::K_BYTES;
  uint64_t *bars = (uint64_t *)(q_s + 2 * Sh::Q_STAGE);
  uint64_t *k_full = bars, *q_full = k_full + 1, *q_empty = q_full + 2, *s_full = q_empty + 2, *s_free = s_full + 2;
  uint32_t *tmem_base_p = (uint32_t *)(s_free + 2);
  volatile int *abort_flag = (volatile int *)(tmem_base_p + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, h = blockIdx.y, kvh = h / a.G;
  if (threadIdx.x == 0) {
    mbar_init(k_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(q_full + s, 1); mbar_init(q_empty + s, 1); mbar_init(s_full + s, 1); mbar_init(s_free + s, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_p)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_p;
  pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) trace_stamp(TR_k_colsum);

  const int n = a.n;
  const int j0 = a.key0 + tile * CS_KEYS;                   // first key of this tile; rows before it see none of its keys
  const int n_steps = n > j0 ? (n - j0 + NQ - 1) / NQ : 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n_steps > 0) {
      const uint64_t pol = policy_evict_first();
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
      mbar_expect_tx(k_full, (uint32_t)Sh::K_BYTES);
      const int sub_rows = min(64, a.page_tokens), n_sub = CS_KEYS / sub_rows;
      for (int sb = 0; sb < n_sub; ++sb) {
        const int j = min(j0 + sb * sub_rows, a.pages_per_seq * a.page_tokens - sub_rows);
        const int pg = a.page_table[a.seq * a.pages_per_seq + (j >> a.page_shift)];
        const int row = (pg * a.hkv + kvh) * a.page_tokens + (j & (a.page_tokens - 1));
        for (int kp = 0; kp < KP; ++kp)
          tma_load_2d(k_s + kp * (CS_KEYS * 128) + sb * sub_rows * 128, &map_k, k_full, kp * 64, row, pol);
      }
      for (int t = 0; t < n_steps; ++t) {
        const int st = t & 1, use = t >> 1;
        if (use >= 1 && !mbar_wait(q_empty + st, (uint32_t)(use - 1) & 1u)) { atomicMax(a.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; break; }
        if (*abort_flag) break;
        mbar_expect_tx(q_full + st, (uint32_t)Sh::Q_STAGE);
        for (int pl = 0; pl < 2; ++pl)
          for (int kp = 0; kp < KP; ++kp)
            tma_load_4d(q_s + st * Sh::Q_STAGE + (pl * KP + kp) * (NQ * 128), &map_q, q_full + st, kp * 64, pl, h, j0 + t * NQ, pol);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: S^T = K Q_hi^T + K Q_lo^T
    if (lane == 0 && n_steps > 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NQ >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      bool ok = mbar_wait(k_full, 0);
      for (int t = 0; t < n_steps && ok; ++t) {
        const int st = t & 1, use = t >> 1;
        if (!mbar_wait(q_full + st, (uint32_t)use & 1u) || (use >= 1 && !mbar_wait(s_free + st, (uint32_t)(use - 1) & 1u))) { ok = false; break; }
        tc_fence_after();
        uint32_t acc = 0u;
        for (int pl = 0; pl < 2; ++pl)
          for (int kp = 0; kp < KP; ++kp) {
            const uint64_t ad = smem_desc(smem_u32(k_s + kp * (CS_KEYS * 128)));
            const uint64_t bd = smem_desc(smem_u32(q_s + st * Sh::Q_STAGE + (pl * KP + kp) * (NQ * 128)));
#pragma unroll
            for (int k = 0; k < 4; ++k) { mma_bf16(tmem_base + (uint32_t)(st * NQ), ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, acc); acc = 1u; }
          }
        mma_commit(q_empty + st);
        mma_commit(s_full + st);
      }
      if (!ok) { atomicMax(a.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ------------------------------------------------------------------ one key (column of the attention matrix) per thread
    const int q = warp & 3;                                   // TMEM lane quarter this warp may access
    const int j = j0 + q * 32 + lane, jv = j - a.vis_start;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const int i_min = j + (a.include_self ? 0 : 1);          // first row whose attention to key j counts
    const float scale = a.scale_log2;
    const float *lse_h = a.lse + (long long)h * n;
    float hs = 0.f;
    bool ok = true;
#pragma unroll 1
    for (int t = 0; t < n_steps && ok; ++t) {
      const int st = t & 1, i0 = j0 + t * NQ;
      int w_ok = 1;
      if (lane == 0) w_ok = mbar_wait(s_full + st, (uint32_t)(t >> 1) & 1u) ? 1 : 0;
      w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
      if (!w_ok || *abort_flag) { ok = false; break; }
      tc_fence_after();
#pragma unroll 1
      for (int c0 = 0; c0 < NQ; c0 += 32) {
        uint32_t sr[32];
        tmem_ld32(lane_addr + (uint32_t)(st * NQ + c0), sr);
        const int il = i0 + c0 + lane;                       // this lane fetches one row's log-sum-exp for the warp
        const float my_l = il < n ? lse_h[il] * 1.4426950408889634f : 0.f;
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int i = i0 + c0 + c;
          const float l2 = __shfl_sync(0xffffffffu, my_l, c);
          const float p = exp2f(__uint_as_float(sr[c]) * scale - l2);
          hs += (i >= i_min && i < n) ? p : 0.f;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_free + st);
    }
    if (n_steps > 0 && !ok && lane == 0) { atomicMax(a.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; }
    if (ok && jv >= 0 && jv < a.v) a.part[(long long)h * a.v + jv] = hs;
  }
  pdl_trigger();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

template <int HD>
static inline const char *colsum_tc_setup() {
  if (cudaFuncSetAttribute(k_colsum_tc<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CsShape<HD>::SMEM) != cudaSuccess)
    return "cannot raise the importance kernel's shared memory limit";
  return nullptr;
}

// Enqueue one launch: grid (key tiles, H).
template <int HD>
static inline cudaError_t colsum_tc_launch(cudaStream_t stream, int use_pdl, const CUtensorMap &mq, const CUtensorMap &mk,
                                           const ColsumTcArgs &a, int n_tiles) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_tiles, a.H, 1); cfg.blockDim = dim3(CS_THREADS);
  cfg.dynamicSmemBytes = CsShape<HD>::SMEM; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = use_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, k_colsum_tc<HD>, mq, mk, a);
}
