// Few-query attention on the tcgen05 tensor cores for sm_100a: the tree-masked verification
// over the paged target cache (Section 3.1), the draft's self- and cross-attention over its flat
// caches (Eq. 1), and the causal prefill attention with the row entropies of Eq. 2.
//
// A CTA owns one tile of 64 query entries (entry = (row, query head of one KV-head group)), one KV
// head and one chunk of keys.  Queries carry ~16 mantissa bits as a high and a low bf16 row, so
// the tile is the MMA's M = 128: row 2e = high part of entry e, row 2e + 1 = its low part; the two
// accumulator lanes of an entry are added with one shuffle.  Keys are walked in blocks of 64,
// GROUP blocks (one group) at a time:
//   S = Q K^T            one chain of tcgen05.mma 128 x (64 x blocks) x 16 over head_dim for the whole
//                        group, A = Q and B = K from shared memory (K-major, 128-byte swizzle,
//                        TMA-fed; the group's K blocks are contiguous), fp32 accumulators in TMEM;
//   softmax              four warps, one TMEM lane per thread; the two lanes of an entry split each
//                        32-key piece between them.  A first pass over the group's S for the row
//                        maximum, a second pass for P = 2^(s - m) (masked) and the row sum; P's high
//                        bf16 part goes to the entry's even row and its low part to the odd row of a
//                        shared-memory tile in the operand layout.  Between groups the O accumulator
//                        is rescaled in TMEM (tcgen05.ld / tcgen05.st);
//   O += P_b V_b         tcgen05.mma 128 x head_dim x 16 steps over each block's keys, A = P_b (K-major)
//                        and B = V_b as stored ([key][head_dim]: an MN-major operand).
// K/V blocks arrive through two TMA rings; during verification the blocks below the verified prefix
// length are requested before the grid dependency resolves.  Flat draft caches carry a low plane
// per key, which costs one more MMA per step.  A chunk leaves (m, l, O) partials for
// k_attn_combine, or the finished rows (and, for the prefill, each row's log-sum-exp and entropy)
// when it is the only chunk.  Warp roles: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..5 =
// softmax and epilogue.  The softmax loops are kept compact on purpose: this kernel's code is
// fetched anew at almost every launch (the weight stream between two launches pushes it out of the
// caches), and straight-line code then costs its own fetch (a fully unrolled version of the same
// loops ran four times slower).  Every mbarrier wait is bounded; on expiry the kernel raises the
// status word and leaves.
#pragma once
#include <map>
#include <vector>

#include "attn_merge.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "rows.cuh"

#define AT_THREADS 192
#define AT_KBLK 64
#define AT_QTILE (128 * 64 * 2)        // one 64-column panel of the query tile (128 rows)
#define AT_KVTILE (64 * 64 * 2)        // one 64-column panel of a 64-key block
#define AT_PTILE (128 * 64 * 2)        // probabilities of one block (128 rows x 64 keys)

enum { AT_VERIFY = 0, AT_DRAFT = 1, AT_PREFILL = 2 };

// Blocks per group: what the shared-memory rings (K and V blocks stay until their MMAs ran) and
// the 512 TMEM columns (head_dim for O, 64 per S_b) hold.
template <int HD, bool FLAT> struct AtShape {
  static constexpr int PLANES = FLAT ? 2 : 1;
  // head_dim 64 over the paged cache takes three blocks, so that O and S fit 256 TMEM columns and two
  // CTAs share an SM (98 KB of shared memory each): twice the key chunks in flight per layer
  // head_dim 128 over the paged cache takes five (231 KB of the 227 KiB a CTA may hold, 448 TMEM columns):
  // prefixes up to 1280 keys then stay one group per chunk when the sequence is cut four ways
  static constexpr int GROUP = HD == 64 ? (FLAT ? 4 : 3) : (HD == 128 ? (FLAT ? 2 : 5) : (FLAT ? 1 : 2));
  static constexpr int TMEM_COLS = HD + GROUP * 64 <= 256 ? 256 : 512;
  static constexpr int CTAS_PER_SM = HD == 64 && !FLAT ? 2 : 1;
  static constexpr int KP = HD / 64;                                 // 64-column panels per row
  static constexpr int KV_STAGE = PLANES * KP * AT_KVTILE;           // one block of K (or of V)
  static constexpr int Q_BYTES = KP * AT_QTILE;
  static constexpr size_t SMEM = 1024 + Q_BYTES + 2 * GROUP * KV_STAGE + 2 * AT_PTILE + 1024;
};

struct AttnTcArgs {
  int mode;                         // AT_*
  int slot_seq[DREAM_MAX_BATCH];    // sequence of each grid-z slot
  const int *prefix_len;            // by sequence: keys [0, prefix) are visible to every row (verify, draft)
  const int *row_in;                // [R] or null: rows with a negative entry are idle; index into anc (draft)
  const int *row_vis;               // [R] or null (draft): an entry >= 0 makes the row see keys [0, entry) and no tail key
  const uint32_t *mask;             // [R][4] visible tail keys (verify)
  const unsigned long long *anc;    // [seq][anc_stride] ancestor-or-self bits over tail keys (draft)
  int anc_stride, strict;
  int rows_per_seq, tail_len, H, G; // query rows per sequence slot, tail keys, query heads, heads per KV head
  int n_keys;                       // prefill: keys in the sequence (row i sees keys 0..i)
  float scale_log2;
  int n_chunks, blocks_per_chunk, n_rt;
  float *part_o, *part_ml;          // [slot][chunk][kvh][rt][64][hd], [..][64][2]
  void *out;                        // [R][H*hd] rows in GEMM-input layout
  XLayout lay;
  int out_chunk_rows;               // prefill: the output rows are laid out per chunk of this many rows ...
  long long out_chunk_stride;       // ... this many elements apart (0: one chunk)
  float *lse, *ent;                 // prefill: [H][n] row log-sum-exp and entropy, or null
  float *row_ent;                   // verify: [R][H] entropy of every tree row's attention distribution, or null
  float *part_u;                    // ... and, with several chunks, the chunks' u = sum p (s - m) beside part_ml
  L2Prefetch next_w;
  // where the K/V blocks live, as rows of the K and V tensor maps
  const int *page_table;            // paged: [max_batch][pages_per_seq]
  int pages_per_seq, page_tokens, page_shift, hkv;
  long long flat_rows_per_head;     // flat: cap (rows per (sequence, K|V, KV head))
  int *status;
};

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z, int w, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w), "l"(policy) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
        "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
        "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Makes this thread's shared-memory stores visible to the asynchronous proxy (the MMA reads P through it).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory descriptor of an MN-major operand with 128-byte swizzle: 64 elements of the MN axis
// are contiguous (one 128-byte row per K index), 8 K-rows form a 1024-byte group, and the next 64
// MN elements start lbo_bytes further on.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t saddr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)(lbo_bytes >> 4) << 16;          // leading byte offset: between 64-element MN blocks
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: between groups of 8 K-rows
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

template <int HD, bool FLAT>
__global__ void __launch_bounds__(AT_THREADS, (AtShape<HD, FLAT>::CTAS_PER_SM))
k_attn_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
          const __grid_constant__ AttnTcArgs a) {
  using Sh = AtShape<HD, FLAT>;
  constexpr int GROUP = Sh::GROUP, KP = Sh::KP, PLANES = Sh::PLANES;
  extern __shared__ uint8_t at_smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)at_smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t *q_s = smem, *k_s = q_s + Sh::Q_BYTES, *v_s = k_s + GROUP * Sh::KV_STAGE, *p_s = v_s + GROUP * Sh::KV_STAGE;
  uint64_t *bars = (uint64_t *)(p_s + 2 * AT_PTILE);
  uint64_t *q_full = bars, *k_full = q_full + 1, *k_empty = k_full + 8, *v_full = k_empty + 8, *v_empty = v_full + 8;
  uint64_t *s_full = v_empty + 8, *s_free = s_full + 8, *p_full = s_free + 8, *p_empty = p_full + 2, *o_done = p_empty + 2;
  uint32_t *tmem_base_p = (uint32_t *)(o_done + 1);
  volatile int *abort_flag = (volatile int *)(tmem_base_p + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, kvh = blockIdx.y / a.n_rt, rt = blockIdx.y - kvh * a.n_rt, slot = blockIdx.z;
  const int seq = a.slot_seq[slot];
  if (warp == 0) {      // a lane per ring stage: the set-up is a few instructions deep instead of a loop
    if (lane < GROUP) {
      mbar_init(k_full + lane, 1); mbar_init(k_empty + lane, 1); mbar_init(v_full + lane, 1); mbar_init(v_empty + lane, 1);
      mbar_init(s_full + lane, 1); mbar_init(s_free + lane, 4);
    } else if (lane >= 8 && lane < 10) { mbar_init(p_full + lane - 8, 4); mbar_init(p_empty + lane - 8, 1); }
    else if (lane == 16) { mbar_init(q_full, 1); mbar_init(o_done, 1); *abort_flag = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_p)), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  l2_prefetch_slice(a.next_w, blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z), gridDim.x * gridDim.y * gridDim.z);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_p;
  // Verification reads the verified prefix and its length, which were written rounds ago (hundreds
  // of kernels back in the stream): its K/V blocks below the prefix length are fetched before the
  // grid dependency resolves.  Everything else is an output of the immediate predecessors.
  const bool early = a.mode == AT_VERIFY;
  if (!early) pdl_wait();

  // ---- the chunk's blocks
  const int rows_total = a.rows_per_seq * a.G;              // entries of this sequence slot
  const int e_base = rt * 64;                               // first entry of the tile
  int total_keys, P = 0;
  if (a.mode == AT_PREFILL) {
    // causal: nothing beyond the tile's last row is visible to any of its rows
    int last_node = min(rows_total - 1, e_base + 63) / a.G;
    total_keys = min(a.n_keys, last_node + 1);
  } else {
    P = a.prefix_len[seq];
    total_keys = P + a.tail_len;
  }
  const int nb = (total_keys + AT_KBLK - 1) / AT_KBLK;
  const int b0 = chunk * a.blocks_per_chunk, b1 = min(nb, b0 + a.blocks_per_chunk);
  const int n_blk = max(0, b1 - b0);

  // K and V of the chunk's block `it` into ring stage it % GROUP (producer thread only)
  const uint64_t pol_kv = policy_evict_first();
  auto issue_kv = [&](int it) {
    const int st = it % GROUP, j0 = (b0 + it) * AT_KBLK;
    // K: [plane][panel][stage][64 keys], so the blocks of a group form one operand of 64 x blocks keys
    uint8_t *kd = k_s + st * AT_KVTILE, *vd = v_s + st * Sh::KV_STAGE;
    constexpr int KSTEP = GROUP * AT_KVTILE;                 // bytes between consecutive (plane, panel) of K
    mbar_expect_tx(k_full + st, (uint32_t)Sh::KV_STAGE);
    mbar_expect_tx(v_full + st, (uint32_t)Sh::KV_STAGE);
    if (FLAT) {
      // rows of the map: (sequence, K | V, KV head, key); the second coordinate selects the plane
      const long long rk = (((long long)seq * 2 + 0) * a.hkv + kvh) * a.flat_rows_per_head + j0;
      const long long rv = (((long long)seq * 2 + 1) * a.hkv + kvh) * a.flat_rows_per_head + j0;
      for (int pl = 0; pl < PLANES; ++pl)
        for (int kp = 0; kp < KP; ++kp) {
          tma_load_3d(kd + (pl * KP + kp) * KSTEP, &map_k, k_full + st, kp * 64, pl, (int)rk, pol_kv);
          tma_load_3d(vd + (pl * KP + kp) * AT_KVTILE, &map_v, v_full + st, kp * 64, pl, (int)rv, pol_kv);
        }
    } else {
      const int sub_rows = min(64, a.page_tokens), n_sub = 64 / sub_rows;
      for (int sb = 0; sb < n_sub; ++sb) {
        const int j = min(j0 + sb * sub_rows, a.pages_per_seq * a.page_tokens - 1);
        const int pg = a.page_table[seq * a.pages_per_seq + (j >> a.page_shift)];
        const int row = (pg * a.hkv + kvh) * a.page_tokens + (j & (a.page_tokens - 1));
        for (int kp = 0; kp < KP; ++kp) {
          tma_load_2d(kd + kp * KSTEP + sb * sub_rows * 128, &map_k, k_full + st, kp * 64, row, pol_kv);
          tma_load_2d(vd + kp * AT_KVTILE + sb * sub_rows * 128, &map_v, v_full + st, kp * 64, row, pol_kv);
        }
      }
    }
  };
  int n_pre = 0;                                            // blocks of the first group already under way
  if (early) {
    if (threadIdx.x == 0 && n_blk > 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
      while (n_pre < min(n_blk, GROUP) && (b0 + n_pre + 1) * AT_KBLK <= P) { issue_kv(n_pre); ++n_pre; }
    }
    pdl_wait();
  }
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) trace_stamp(TR_k_attn_tc);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n_blk > 0) {
      const uint64_t pol_q = policy_evict_last();
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
      // queries: box (64 columns, high | low, G heads, 64 / G rows) -> row 2 e + part of the tile
      mbar_expect_tx(q_full, (uint32_t)Sh::Q_BYTES);
      const int node0 = slot * a.rows_per_seq + e_base / a.G;
      for (int kp = 0; kp < KP; ++kp) tma_load_4d(q_s + kp * AT_QTILE, &map_q, q_full, kp * 64, 0, kvh * a.G, node0, pol_q);
      for (int it = n_pre; it < n_blk; ++it) {
        const int st = it % GROUP, use = it / GROUP;
        if (use >= 1 && (!mbar_wait(k_empty + st, (uint32_t)(use - 1) & 1u) || !mbar_wait(v_empty + st, (uint32_t)(use - 1) & 1u))) {
          atomicMax(a.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; break;
        }
        if (*abort_flag) break;
        issue_kv(it);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n_blk > 0) {
      // fp32 accumulate, bf16 operands, M = 128; S: N = 64, both K-major; O: N = head_dim, B MN-major
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t o_addr = tmem_base, s_addr0 = tmem_base + HD;
      bool ok = mbar_wait(q_full, 0);
      const int n_groups = (n_blk + GROUP - 1) / GROUP;
      for (int gi = 0; gi < n_groups && ok; ++gi) {
        const int gb = gi * GROUP, ge = min(n_blk, gb + GROUP);
        // S = Q K^T for all keys of the group at once: N = 64 x blocks
        for (int it = gb; it < ge && ok; ++it) {
          const int st = it % GROUP;
          if (!mbar_wait(k_full + st, (uint32_t)gi & 1u) || (gi >= 1 && !mbar_wait(s_free + st, (uint32_t)(gi - 1) & 1u))) ok = false;
        }
        if (!ok) break;
        tc_fence_after();
        // (an MMA's N ends at 256: a group of five blocks takes a chain of four blocks and one of one)
        for (int b0 = 0; b0 < ge - gb; b0 += 4) {
          const uint32_t n_keys_g = (uint32_t)min(4, ge - gb - b0) * 64u;
          const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((n_keys_g >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
          uint32_t acc = 0u;
          for (int pl = 0; pl < PLANES; ++pl)
            for (int kp = 0; kp < KP; ++kp) {
              const uint64_t ad = smem_desc(smem_u32(q_s + kp * AT_QTILE));
              const uint64_t bd = smem_desc(smem_u32(k_s + ((pl * KP + kp) * GROUP + b0) * AT_KVTILE));
#pragma unroll
              for (int k = 0; k < 4; ++k) { mma_bf16(s_addr0 + (uint32_t)(b0 * 64), ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc_s, acc); acc = 1u; }
            }
        }
        for (int it = gb; it < ge; ++it) { mma_commit(k_empty + it % GROUP); mma_commit(s_full + it % GROUP); }
        for (int it = gb; it < ge && ok; ++it) {                       // O += P_b V_b
          const int st = it % GROUP, pb = it & 1;
          if (!mbar_wait(p_full + pb, (uint32_t)(it >> 1) & 1u) || !mbar_wait(v_full + st, (uint32_t)gi & 1u)) { ok = false; break; }
          tc_fence_after();
          const uint64_t ad = smem_desc(smem_u32(p_s + pb * AT_PTILE));
          for (int pl = 0; pl < PLANES; ++pl) {
            const uint64_t bd = smem_desc_mn(smem_u32(v_s + st * Sh::KV_STAGE + pl * KP * AT_KVTILE), AT_KVTILE);
#pragma unroll
            for (int k = 0; k < 4; ++k)                                 // 16 keys = two groups of 8 K-rows = 2048 bytes
              mma_bf16(o_addr, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 128), idesc_o, (it > 0 || pl > 0 || k > 0) ? 1u : 0u);
          }
          mma_commit(p_empty + pb);
          mma_commit(v_empty + st);
          if (it == ge - 1) mma_commit(o_done);
        }
      }
      if (!ok) { atomicMax(a.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ------------------------------------------------------------------ softmax and epilogue: one row per thread
    const int q = warp & 3;                                   // TMEM lane quarter this warp may access
    const int row = q * 32 + lane, e = e_base + (row >> 1), part = row & 1;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    // what this row sees: keys below `vis_end`, plus tail key j (key index tail0 + j) for the bits of mw
    int r = -1, h = 0, vis_end = 0, tail0 = 0;
    uint32_t mw[4] = {0u, 0u, 0u, 0u};
    if (e < rows_total) {
      const int node = e / a.G;
      r = slot * a.rows_per_seq + node; h = kvh * a.G + (e - node * a.G);
      if (a.mode == AT_PREFILL) vis_end = node + 1;
      else {
        vis_end = P; tail0 = P;
        if (a.mode == AT_VERIFY) {
          for (int wd = 0; wd < 4; ++wd) mw[wd] = a.mask[(long long)r * 4 + wd];
        } else {
          const int in = a.row_in ? a.row_in[r] : 0;
          const int rv = a.row_vis ? a.row_vis[r] : -1;
          if (rv >= 0) vis_end = rv;
          else if (in < 0) r = -1;
          else {
            unsigned long long bits = a.anc[(long long)seq * a.anc_stride + in];
            if (a.strict) bits &= ~(1ull << in);
            mw[0] = (uint32_t)bits; mw[1] = (uint32_t)(bits >> 32);
          }
        }
      }
    }
    // Everything the loops below read sits in registers (the argument block is read through memory),
    // and the loops are kept small on purpose: the kernel's code is fetched anew at every launch
    // (the weight stream has pushed it out of L2 by then), so straight-line code costs its fetch.
    const float scale = a.scale_log2;
    const int tail_len = a.mode == AT_PREFILL ? 0 : a.tail_len;
    const unsigned long long mlo = (unsigned long long)mw[0] | ((unsigned long long)mw[1] << 32),
                             mhi = (unsigned long long)mw[2] | ((unsigned long long)mw[3] << 32);
    // visibility of the 32 keys j32 .. j32 + 31 as a bit mask
    auto vis32 = [=](int j32) -> uint32_t {
      const int npre = min(32, max(0, vis_end - j32));
      uint32_t m = npre >= 32 ? 0xffffffffu : (1u << npre) - 1u;
      if (npre < 32 && tail_len > 0) {
        const int sh = j32 - tail0;                            // tail key index of bit 0
        unsigned long long t;
        if (sh < 0) t = sh > -32 ? mlo << (-sh) : 0ull;
        else if (sh < 64) t = (mlo >> sh) | (sh ? mhi << (64 - sh) : 0ull);
        else t = sh < 128 ? mhi >> (sh - 64) : 0ull;
        m |= (uint32_t)t;
      }
      return m;
    };
    float m_run = -INFINITY, l_run = 0.f, u_run = 0.f;       // exp2 domain; u = sum p (s - m) for the entropy
    const bool want_ent = a.ent != nullptr || a.row_ent != nullptr;
    bool ok = n_blk > 0;
    const int n_groups = (n_blk + GROUP - 1) / GROUP;
#pragma unroll 1
    for (int gi = 0; gi < n_groups && ok; ++gi) {
      const int gb = gi * GROUP, ge = min(n_blk, gb + GROUP);
      // ---- first pass: the row maximum over the group's keys
      float gmax = m_run;
#pragma unroll 1
      for (int it = gb; it < ge && ok; ++it) {
        const int st = it % GROUP, j0 = (b0 + it) * AT_KBLK;
        int w_ok = 1;
        if (lane == 0) w_ok = mbar_wait(s_full + st, (uint32_t)gi & 1u) ? 1 : 0;
        w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
        if (!w_ok || *abort_flag) { ok = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t sr[32];
          tmem_ld32(lane_addr + (uint32_t)(HD + st * 64 + ch * 32), sr);
          const uint32_t vm = vis32(j0 + ch * 32);
          tmem_ld_wait();
          // lanes 2e and 2e+1 hold the products of entry e's high and low query parts: the even lane
          // keeps keys 0..15 of the chunk and the odd lane 16..31, each sends the partner what it needs
          const uint32_t vmh = vm >> (part * 16);
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const float send = __uint_as_float(part ? sr[c] : sr[16 + c]);
            const float mine = __uint_as_float(part ? sr[16 + c] : sr[c]);
            const float t = (mine + __shfl_xor_sync(0xffffffffu, send, 1)) * scale;
            gmax = fmaxf(gmax, ((vmh >> c) & 1u) ? t : -INFINITY);
          }
        }
      }
      gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, 1));
      if (!ok) break;
      const float base = gmax == -INFINITY ? 0.f : gmax;
      const float corr = exp2f(m_run - base);                 // 0 when nothing was seen before
      if (gi >= 1) {
        // ---- the accumulator of the earlier groups takes the new maximum
        int w_ok = 1;
        if (lane == 0) w_ok = mbar_wait(o_done, (uint32_t)(gi - 1) & 1u) ? 1 : 0;
        w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
        if (!w_ok) { ok = false; break; }
        tc_fence_after();
        if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll 1
          for (int c0 = 0; c0 < HD; c0 += 32) {
            uint32_t orr[32];
            tmem_ld32(lane_addr + (uint32_t)c0, orr);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * corr);
            tmem_st32(lane_addr + (uint32_t)c0, orr);
          }
          tmem_st_wait();
        }
        if (want_ent) u_run = l_run > 0.f ? corr * (u_run - (base - m_run) * l_run) : 0.f;
        l_run *= corr;
      }
      m_run = gmax;
      // ---- second pass: probabilities, row sum, P's high or low part into shared memory
#pragma unroll 1
      for (int it = gb; it < ge && ok; ++it) {
        const int st = it % GROUP, pb = it & 1, j0 = (b0 + it) * AT_KBLK;
        if ((it >> 1) >= 1) {
          int w_ok = 1;
          if (lane == 0) w_ok = mbar_wait(p_empty + pb, (uint32_t)((it >> 1) - 1) & 1u) ? 1 : 0;
          w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
          if (!w_ok || *abort_flag) { ok = false; break; }
        }
        uint8_t *prow0 = p_s + pb * AT_PTILE;
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t sr[32];
          tmem_ld32(lane_addr + (uint32_t)(HD + st * 64 + ch * 32), sr);
          const uint32_t vm = vis32(j0 + ch * 32);
          tmem_ld_wait();
          const uint32_t vmh = vm >> (part * 16);
          uint32_t ph[8], pl2[8];
#pragma unroll
          for (int c = 0; c < 16; c += 2) {
            const float s0 = __uint_as_float(part ? sr[c] : sr[16 + c]), s1 = __uint_as_float(part ? sr[c + 1] : sr[17 + c]);
            const float m0 = __uint_as_float(part ? sr[16 + c] : sr[c]), m1 = __uint_as_float(part ? sr[17 + c] : sr[c + 1]);
            const float d0 = (m0 + __shfl_xor_sync(0xffffffffu, s0, 1)) * scale - base;
            const float d1 = (m1 + __shfl_xor_sync(0xffffffffu, s1, 1)) * scale - base;
            const float p0 = ((vmh >> c) & 1u) ? exp2f(d0) : 0.f, p1 = ((vmh >> (c + 1)) & 1u) ? exp2f(d1) : 0.f;
            l_run += p0 + p1;
            if (want_ent) u_run += (p0 > 0.f ? p0 * d0 : 0.f) + (p1 > 0.f ? p1 * d1 : 0.f);
            split_pair(p0, p1, ph[c >> 1], pl2[c >> 1]);
          }
          // this lane's 16 keys: high parts into the entry's even row, low parts into its odd row; 16-byte
          // pieces swizzled like the MMA expects a K-major operand (piece ^ (row & 7))
          uint8_t *row_hi = prow0 + (row & ~1) * 128, *row_lo = row_hi + 128;
#pragma unroll
          for (int pc = 0; pc < 2; ++pc) {
            const int piece = ch * 4 + part * 2 + pc;
            *reinterpret_cast<uint4 *>(row_hi + ((piece ^ (row & 6)) << 4)) = make_uint4(ph[pc * 4], ph[pc * 4 + 1], ph[pc * 4 + 2], ph[pc * 4 + 3]);
            *reinterpret_cast<uint4 *>(row_lo + ((piece ^ ((row & 6) | 1)) << 4)) = make_uint4(pl2[pc * 4], pl2[pc * 4 + 1], pl2[pc * 4 + 2], pl2[pc * 4 + 3]);
          }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) { mbar_arrive(p_full + pb); mbar_arrive(s_free + st); }
      }
    }
    // ---- epilogue: the row's accumulator (lanes 2e and 2e+1 added), partial or finished
    if (ok) {
      int w_ok = 1;
      if (lane == 0) w_ok = mbar_wait(o_done, (uint32_t)(n_groups - 1) & 1u) ? 1 : 0;
      w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
      ok = w_ok != 0;
    }
    if (n_blk > 0 && !ok && lane == 0) { atomicMax(a.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; }
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);           // each lane of a pair summed half of the keys
    u_run += __shfl_xor_sync(0xffffffffu, u_run, 1);
    pdl_trigger();                                            // the keys are done: the kernel that follows may take the SMs
    if (n_blk == 0 || ok) {
      tc_fence_after();
      const int Hkv = a.H / a.G;
      const long long pbase = ((((long long)slot * a.n_chunks + chunk) * Hkv + kvh) * a.n_rt + rt) * 64 + (row >> 1);
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t orr[32];
        if (n_blk > 0) { tmem_ld32(lane_addr + (uint32_t)c0, orr); tmem_ld_wait(); }
        else {
#pragma unroll
          for (int c = 0; c < 32; ++c) orr[c] = 0u;
        }
        // the even lane keeps columns 0..15 of the chunk, the odd lane 16..31 (as in the GEMM's epilogue)
        float v[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const float send = __uint_as_float(part ? orr[c] : orr[16 + c]);
          const float mine = __uint_as_float(part ? orr[16 + c] : orr[c]);
          v[c] = mine + __shfl_xor_sync(0xffffffffu, send, 1);
        }
        if (r < 0) continue;
        const int col = c0 + part * 16;
        if (a.n_chunks == 1) {
          bf16 *out = reinterpret_cast<bf16 *>(a.out);
          long long o = a.out_chunk_stride ? (long long)(r / a.out_chunk_rows) * a.out_chunk_stride + (long long)(r % a.out_chunk_rows) * a.lay.row_stride
                                           : (long long)r * a.lay.row_stride;
#pragma unroll
          for (int c = 0; c < 16; c += 4)
            store_split4<bf16>(out + o + h * HD + col + c, a.lay.lo_delta, make_float4(v[c] * inv, v[c + 1] * inv, v[c + 2] * inv, v[c + 3] * inv));
        } else {
          float *po = a.part_o + pbase * HD + col;
#pragma unroll
          for (int c = 0; c < 16; c += 4) *reinterpret_cast<float4 *>(po + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
        }
      }
      if (r >= 0 && part == 0) {
        if (a.n_chunks > 1) {
          *reinterpret_cast<float2 *>(a.part_ml + pbase * 2) = make_float2(m_run, l_run);
          if (a.row_ent) a.part_u[pbase] = u_run;
        } else if (a.row_ent) {
          a.row_ent[(long long)r * a.H + h] = l_run > 0.f ? logf(l_run) - u_run * 0.6931471805599453f / l_run : 0.f;
        }
        if (a.lse) {
          // natural-log units: lse = m ln 2 + ln l;  H = ln l - u ln 2 / l
          const int node = r - slot * a.rows_per_seq;
          const float ln2 = 0.6931471805599453f;
          a.lse[(long long)h * a.n_keys + node] = m_run * ln2 + logf(l_run);
          if (a.ent) a.ent[(long long)h * a.n_keys + node] = logf(l_run) - u_run * ln2 / l_run;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ host side

// Tensor maps of the attention operands, cached by everything that defines them.
struct AtMapCache { std::map<std::vector<unsigned long long>, CUtensorMap> maps; };

// bf16 tensor of `rank` dimensions (innermost first), 128-byte swizzle, zero fill beyond the extents.
static inline bool at_map(GemmTcPlan *pl, AtMapCache *cache, const void *ptr, int rank, const unsigned long long *dims,
                          const unsigned long long *strides_bytes, const unsigned *box, CUtensorMap *out) {
  std::vector<unsigned long long> key;
  key.push_back((unsigned long long)(uintptr_t)ptr);
  key.push_back((unsigned long long)rank);
  for (int i = 0; i < rank; ++i) { key.push_back(dims[i]); key.push_back(box[i]); if (i) key.push_back(strides_bytes[i - 1]); }
  auto it = cache->maps.find(key);
  if (it != cache->maps.end()) { *out = it->second; return true; }
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; if (i) st[i - 1] = strides_bytes[i - 1]; }
  CUtensorMap m;
  CUresult r = pl->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(ptr), d, st, b, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache->maps.size() > 4096) cache->maps.clear();
  cache->maps[key] = m;
  *out = m;
  return true;
}

template <int HD, bool FLAT>
static inline const char *attn_tc_setup() {
  if (cudaFuncSetAttribute(k_attn_tc<HD, FLAT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AtShape<HD, FLAT>::SMEM) != cudaSuccess)
    return "cannot raise the attention kernel's shared memory limit";
  return nullptr;
}

// Enqueue one attention launch: grid (a.n_chunks, H_kv * a.n_rt, n_slots).
template <int HD, bool FLAT>
static inline cudaError_t attn_tc_launch(cudaStream_t stream, int use_pdl, const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv,
                                         const AttnTcArgs &a, int n_slots) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.n_chunks, (a.H / a.G) * a.n_rt, n_slots); cfg.blockDim = dim3(AT_THREADS);
  cfg.dynamicSmemBytes = AtShape<HD, FLAT>::SMEM; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = use_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, k_attn_tc<HD, FLAT>, mq, mk, mv, a);
}
