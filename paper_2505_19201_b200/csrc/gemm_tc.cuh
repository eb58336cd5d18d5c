// Weight-streaming small-M GEMM for sm_100a:  out[t][c] = sum_k X[t][k] * W[c][k].
//
// The token count is tiny (<= 128 rows) and the weight matrix is large, so the kernel is bound
// by streaming W from HBM once.  Design:
//   * tokens are the MMA's M (the 128 TMEM lanes) and 256 weight rows are its N (TMEM columns):
//     one tcgen05.mma (cta_group::1, kind::f16, bf16 x bf16 -> fp32) covers 128 x 256 x 16, so a
//     32 KB weight panel costs four instructions and the issuing thread never limits the stream;
//   * activations carry ~16 mantissa bits as two bf16 rows per token (high and low part):
//       - up to 64 tokens: the rows are interleaved (row 2t = high, row 2t+1 = low), one A tile
//         holds both, and the epilogue adds neighbouring TMEM lanes with one shuffle;
//       - 65..128 tokens: high and low parts are two A tiles and two MMAs per k-step accumulate
//         into the same TMEM columns;
//   * two independent shared-memory rings fed by TMA (cp.async.bulk.tensor.2d, 128-byte swizzle,
//     no multicast): one for W panels (256 rows x 64 k, evict-first) and one for X panels
//     (128 rows x 64 k, served by L2, evict-last);
//   * persistent stream-K: the (tile, panel) units are dealt out in equal contiguous ranges to one
//     CTA per SM; a CTA that covers part of a tile writes a partial sum to its own slot and the
//     consumer adds the slots in a fixed order;
//   * programmatic dependent launch: W never changes, so its ring fills before the grid
//     dependency resolves; only the X producer and the epilogue wait for the previous kernel;
//   * warp roles: 0 = W producer, 1 = MMA issuer and TMEM owner, 6 = X producer, 2..5 and 7..10 =
//     epilogue (tcgen05.ld -> 128-bit stores; the first set drains accumulator columns 0..127, the
//     second 128..255, loads software-pipelined, each chunk turned in shared memory so that a
//     store covers whole 128-byte runs of a row); two TMEM accumulators alternate so that the
//     epilogue of one segment overlaps the MMAs of the next;
//   * every mbarrier wait is bounded: on expiry the kernel raises the status word and leaves.
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <map>
#include <tuple>

#include "common.cuh"

#define TC_BN 256               // weight rows per tile (MMA N)
#define TC_BK 64                // k elements per panel (128 bytes: one swizzle row)
#define TC_THREADS 352          // 11 warps, see the roles above
#define TC_SPIN_LIMIT (1u << 24)
#define TC_WPANEL (TC_BN * TC_BK * 2)
#define TC_STG_LD 36            // floats per row of an epilogue staging tile (32 + padding)
#define TC_STG_BYTES (8 * 16 * TC_STG_LD * 4)
#define TC_XTILE (128 * TC_BK * 2)

enum { TC_X_PLAIN = 0, TC_X_INTERLEAVED = 1, TC_X_PLANAR = 2 };

struct TcParams {
  float *out;
  long long slot_stride;        // floats between partial-sum slots
  int N, K, KB, n_tiles, total_units, upc;
  int n_tok;                    // real token rows
  int x_mode;                   // TC_X_*
  int lo_rows;                  // TC_X_PLANAR: row of the first low part in the X tensor map
  int m_tiles;                  // token tiles of 128 rows per launch: 1, or 2 (TC_X_PLANAR, 129..256 tokens)
  int wp, w_stages, x_stages;   // panels per ring stage, ring depths
  int *status;
};

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait on a phase parity; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
  uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < TC_SPIN_LIMIT; ++it) {
    uint32_t done;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);        // start address
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }


// ------------------------------------------------------------------------------------------ kernel
// Dynamic shared memory (1024-byte aligned): W ring [w_stages][wp][32 KB], X ring
// [x_stages][wp][16 KB, or 32 KB = high tile | low tile when planar], then the barriers.
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const bool planar = p.x_mode == TC_X_PLANAR;
  const uint32_t wstage_bytes = (uint32_t)p.wp * TC_WPANEL;
  const uint32_t xpanel_bytes = planar ? 2u * TC_XTILE * (uint32_t)p.m_tiles : (uint32_t)TC_XTILE;   // per token tile: high | low
  const int n_buf = p.m_tiles == 2 ? 1 : 2;                // two token tiles fill all 512 TMEM columns: one accumulator set
  const uint32_t xstage_bytes = (uint32_t)p.wp * xpanel_bytes;
  uint8_t *wring = smem, *xring = smem + (size_t)p.w_stages * wstage_bytes;
  uint64_t *bars = (uint64_t *)(xring + (size_t)p.x_stages * xstage_bytes);
  uint64_t *full_w = bars, *empty_w = full_w + p.w_stages, *full_x = empty_w + p.w_stages, *empty_x = full_x + p.x_stages;
  uint64_t *acc_full = empty_x + p.x_stages, *acc_empty = acc_full + 2;
  uint32_t *tmem_base_p = (uint32_t *)(acc_empty + 2);
  volatile int *abort_flag = (volatile int *)(tmem_base_p + 1);
  float *stage_tiles = (float *)(bars + 64);               // 8 warps x [16][TC_STG_LD] floats, 512 bytes behind the barriers' start

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (blockIdx.x == 0 && threadIdx.x == 0) trace_stamp(TR_none);     // CTA start, before any dependency
  if (warp == 0) {      // one barrier pair per lane: the set-up is a few instructions deep instead of a loop
    if (lane < p.w_stages) { mbar_init(full_w + lane, 1); mbar_init(empty_w + lane, 1); }
    else if (lane >= 8 && lane < 8 + p.x_stages) { mbar_init(full_x + lane - 8, 1); mbar_init(empty_x + lane - 8, 1); }
    else if (lane >= 16 && lane < 18) { mbar_init(acc_full + lane - 16, 1); mbar_init(acc_empty + lane - 16, 8); }
    else if (lane == 31) *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {      // all 512 TMEM columns (two accumulators of 256), allocated by one full warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_p)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_trigger();
  const uint32_t tmem_base = *tmem_base_p;
  const int u_begin = blockIdx.x * p.upc, u_end = min(u_begin + p.upc, p.total_units);

  if (warp == 0) {
    // ------------------------------------------------------------------ W producer: weights are
    // constant, so nothing here waits for anything but ring space
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
      int s = 0, u = u_begin;
      uint32_t ph = 0;
      bool wrapped = false;
      while (u < u_end) {
        int tile = u / p.KB, kb = u - tile * p.KB;
        int np = min(p.wp, min(p.KB - kb, u_end - u));
        if (wrapped && !mbar_wait(empty_w + s, ph ^ 1)) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; break; }
        if (*abort_flag) break;
        uint8_t *dst = wring + (size_t)s * wstage_bytes;
        mbar_expect_tx(full_w + s, (uint32_t)np * TC_WPANEL);
        for (int q = 0; q < np; ++q) tma_load_2d(dst + (size_t)q * TC_WPANEL, &map_w, full_w + s, (kb + q) * TC_BK, tile * TC_BN, pol);
        u += np;
        if (++s == p.w_stages) { s = 0; ph ^= 1; wrapped = true; }
      }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ X producer: waits until the
    // input exists (previous kernel), then feeds one X stage per W stage
    if (lane == 0) {
      const uint64_t pol = policy_evict_last();
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
      pdl_wait();
      if (blockIdx.x == 0) trace_stamp(TR_k_gemm_tc);
      int s = 0, u = u_begin;
      uint32_t ph = 0;
      bool wrapped = false;
      while (u < u_end) {
        int tile = u / p.KB, kb = u - tile * p.KB;
        int np = min(p.wp, min(p.KB - kb, u_end - u));
        if (wrapped && !mbar_wait(empty_x + s, ph ^ 1)) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; break; }
        if (*abort_flag) break;
        uint8_t *dst = xring + (size_t)s * xstage_bytes;
        mbar_expect_tx(full_x + s, (uint32_t)np * xpanel_bytes);
        for (int q = 0; q < np; ++q) {
          if (!planar) tma_load_2d(dst + (size_t)q * xpanel_bytes, &map_x, full_x + s, (kb + q) * TC_BK, 0, pol);
          else
            for (int mt = 0; mt < p.m_tiles; ++mt) {
              uint8_t *dt = dst + (size_t)q * xpanel_bytes + (size_t)mt * 2 * TC_XTILE;
              tma_load_2d(dt, &map_x, full_x + s, (kb + q) * TC_BK, mt * 128, pol);
              tma_load_2d(dt + TC_XTILE, &map_x, full_x + s, (kb + q) * TC_BK, p.lo_rows + mt * 128, pol);
            }
        }
        u += np;
        if (++s == p.x_stages) { s = 0; ph ^= 1; wrapped = true; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = 256, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TC_BN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      int ws = 0, xs = 0, u = u_begin;
      uint32_t wph = 0, xph = 0, seg = 0;
      bool ok = true;
      while (u < u_end && ok) {
        int tile = u / p.KB;
        int seg_end = min((tile + 1) * p.KB, u_end);
        const int buf = (int)seg % n_buf, use = (int)seg / n_buf;       // use: earlier segments in this accumulator set
        if (use >= 1 && !mbar_wait(acc_empty + buf, (uint32_t)(use - 1) & 1u)) { ok = false; break; }
        tc_fence_after();
        uint32_t d_addr = tmem_base + (uint32_t)buf * TC_BN;
        uint32_t accum = 0u;
        while (u < seg_end) {
          int np = min(p.wp, seg_end - u);
          if (!mbar_wait(full_w + ws, wph) || !mbar_wait(full_x + xs, xph)) { ok = false; break; }
          tc_fence_after();
          uint32_t sw0 = smem_u32(wring + (size_t)ws * wstage_bytes), sx0 = smem_u32(xring + (size_t)xs * xstage_bytes);
          for (int q = 0; q < np; ++q) {
            uint64_t bd = smem_desc(sw0 + (uint32_t)q * TC_WPANEL);
            for (int mt = 0; mt < p.m_tiles; ++mt) {
              const uint32_t xa = sx0 + (uint32_t)q * xpanel_bytes + (uint32_t)mt * 2u * TC_XTILE;
              const uint64_t ad = smem_desc(xa), al = smem_desc(xa + TC_XTILE);
              const uint32_t dm = d_addr + (uint32_t)mt * TC_BN;
              uint32_t acc = accum;
#pragma unroll
              for (int k = 0; k < TC_BK / 16; ++k) {
                mma_bf16(dm, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, acc);
                acc = 1u;
                if (planar) mma_bf16(dm, al + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, 1u);
              }
            }
            accum = 1u;
          }
          mma_commit(empty_x + xs);           // frees both stages once these MMAs have read them
          mma_commit(empty_w + ws);
          u += np;
          if (++ws == p.w_stages) { ws = 0; wph ^= 1; }
          if (++xs == p.x_stages) { xs = 0; xph ^= 1; }
        }
        if (!ok) break;
        mma_commit(acc_full + buf);           // accumulator complete
        ++seg;
      }
      if (!ok) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ------------------------------------------------------------------ warps 2..5, 7..10: epilogue
    // of the CTA's segments (partial sums to this CTA's slot)
    const int q = warp & 3;                   // TMEM lane quarter this warp may read
    const int half = warp >= 7 ? 1 : 0;       // which 128 accumulator columns this warp drains
    const int pwarp = warp < 7 ? warp - 2 : warp - 3;                   // 0..7 among these warps
    float *stg = stage_tiles + pwarp * (16 * TC_STG_LD);                // this warp's staging tile
    pdl_wait();                               // the output buffer belongs to earlier kernels
    const bool inter = p.x_mode == TC_X_INTERLEAVED;
    const int part = inter ? lane & 1 : 0;
    uint32_t seg = 0;
    int u = u_begin;
    while (u < u_end) {
      int tile = u / p.KB;
      int seg_end = min((tile + 1) * p.KB, u_end);
      const int buf = (int)seg % n_buf, use = (int)seg / n_buf;
      int ok = 1;
      if (lane == 0) ok = mbar_wait(acc_full + buf, (uint32_t)use & 1u) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok || *abort_flag) { if (lane == 0) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; } break; }
      tc_fence_after();
      int first_cta = (tile * p.KB) / p.upc;
      int slot = (int)blockIdx.x - first_cta;
      float *dst0 = p.out + (long long)slot * p.slot_stride + tile * TC_BN;       // row 0 of this CTA's slot, first column of the tile
      for (int mt = 0; mt < p.m_tiles; ++mt) {      // token tiles: rows mt * 128 .. of the output, accumulator columns mt * 256 ..
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf + mt) * TC_BN;
      // four chunks of 32 columns; the TMEM load of chunk i+1 is in flight while chunk i is stored.
      // A lane holds values of one row, but a store instruction is cheapest when the lanes of a
      // warp cover whole 128-byte runs of a row: the chunk goes through a [16][32] tile in shared
      // memory (rows padded to 36 floats) and leaves as 4 stores of 4 rows x 128 bytes.
      uint32_t ra[32], rb[32];
      tmem_ld32(taddr + (uint32_t)half * 128u, ra);
#pragma unroll
      for (int ci = 0; ci < 4; ++ci) {
        const int col0 = half * 128 + ci * 32;
        uint32_t (&r)[32] = (ci & 1) ? rb : ra;
        tmem_ld_wait();
        if (ci + 1 < 4) tmem_ld32(taddr + (uint32_t)(col0 + 32), (ci & 1) ? ra : rb);
        const int c4 = (lane & 7) * 4;
        const bool col_ok = tile * TC_BN + col0 + c4 < p.N;
        if (inter) {
          // lanes 2t and 2t+1 hold the products of token t's high and low parts.  The even lane
          // keeps columns 0..15 of the chunk and the odd lane 16..31: each sends the partner
          // the 16 values it needs and adds what it receives to its own.
          float4 *srow = reinterpret_cast<float4 *>(stg + (lane >> 1) * TC_STG_LD + part * 16);
#pragma unroll
          for (int j4 = 0; j4 < 4; ++j4) {
            float v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int j = j4 * 4 + e;
              float send = __uint_as_float(part ? r[j] : r[16 + j]);
              float mine = __uint_as_float(part ? r[16 + j] : r[j]);
              v[e] = mine + __shfl_xor_sync(0xffffffffu, send, 1);
            }
            srow[j4] = make_float4(v[0], v[1], v[2], v[3]);
          }
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int tl = i * 4 + (lane >> 3), tok = q * 16 + tl;
            float4 val = *reinterpret_cast<const float4 *>(stg + tl * TC_STG_LD + c4);
            if (tok < p.n_tok && col_ok) *reinterpret_cast<float4 *>(dst0 + (long long)tok * p.N + col0 + c4) = val;
          }
          __syncwarp();
        } else {
          // one row per lane: two halves of 16 rows through the same tile
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if ((lane >> 4) == h) {
              float4 *srow = reinterpret_cast<float4 *>(stg + (lane & 15) * TC_STG_LD);
#pragma unroll
              for (int j4 = 0; j4 < 8; ++j4)
                srow[j4] = make_float4(__uint_as_float(r[j4 * 4]), __uint_as_float(r[j4 * 4 + 1]), __uint_as_float(r[j4 * 4 + 2]),
                                       __uint_as_float(r[j4 * 4 + 3]));
            }
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int tl = i * 4 + (lane >> 3), tok = mt * 128 + q * 32 + h * 16 + tl;
              float4 val = *reinterpret_cast<const float4 *>(stg + tl * TC_STG_LD + c4);
              if (tok < p.n_tok && col_ok) *reinterpret_cast<float4 *>(dst0 + (long long)tok * p.N + col0 + c4) = val;
            }
            __syncwarp();
          }
        }
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + buf);
      u = seg_end;
      ++seg;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ host side

struct GemmTcPlan {
  PFN_cuTensorMapEncodeTiled_v12000 encode;
  int n_sms;
  int max_smem;
  int use_pdl;
  int *status;
  std::map<std::tuple<const void *, int, int, int>, CUtensorMap> maps;
};

static inline const char *gemm_tc_plan_init(GemmTcPlan *pl, int *status, int use_pdl) {
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn)
    return "cuTensorMapEncodeTiled not available";
  pl->encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&pl->n_sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&pl->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, pl->max_smem) != cudaSuccess)
    return "cannot raise the dynamic shared memory limit";
  pl->status = status;
  pl->use_pdl = use_pdl;
  return nullptr;
}

// Largest token count one launch takes: 64 with interleaved high/low rows, 128 otherwise.
#define TC_ROWS_SPLIT_1MMA 64
#define TC_ROWS_MAX 128

static inline bool gemm_tc_supported(int N, int K) {
  return K % TC_BK == 0 && K >= TC_BK && N % 8 == 0 && N >= 8;
}

// bf16 row-major [rows][K] matrix, box = 64 x box_rows, 128-byte swizzle.  Rows of a box that lie
// beyond `rows` read as zero.
// The encoded map is copied to *out: the cache may drop its entries at any later call.
static inline bool tc_map(GemmTcPlan *pl, const void *ptr, int rows, int K, int box_rows, CUtensorMap *out) {
  auto key = std::make_tuple(ptr, rows, K, box_rows);
  auto it = pl->maps.find(key);
  if (it != pl->maps.end()) { *out = it->second; return true; }
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {TC_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = pl->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (pl->maps.size() > 8192) pl->maps.clear();
  pl->maps[key] = m;
  *out = m;
  return true;
}

// Floats one launch may write when its slots hold slot_rows x N: a tile is shared by at most
// ceil(KB / upc) + 1 CTAs.  n_sms <= 0 gives the bound that holds for any SM count.
static inline long long gemm_tc_out_floats(int n_sms, int slot_rows, int N, int K) {
  int KB = K / TC_BK, n_tiles = (N + TC_BN - 1) / TC_BN;
  long long total = (long long)n_tiles * KB;
  long long slots;
  if (n_sms <= 0) slots = KB + 1;
  else {
    long long grid = n_sms < total ? n_sms : total;
    long long upc = (total + grid - 1) / grid;
    slots = (KB + upc - 1) / upc + 1;
  }
  return slots * (long long)slot_rows * N;
}

// Enqueue one GEMM.
//   X: bf16, row-major, K columns.  TC_X_PLAIN: row t = token t.  TC_X_INTERLEAVED: row 2t = high
//   part of token t, row 2t+1 = low part.  TC_X_PLANAR: row t = high part, row lo_rows + t = low part.
//   rows <= 64 when interleaved, <= 128 otherwise, except that TC_X_PLANAR with lo_rows >= 256 takes
//   up to 256 rows as two token tiles that share every weight panel (the weights stream once;
//   both accumulators fill the TMEM, so epilogues no longer overlap the next segment's MMAs).
//   slot_rows >= rows: rows of a partial-sum slot.
// *g receives the descriptor consumers read the result through.  Returns false if the launch could
// not be made.
static inline bool gemm_tc_launch(GemmTcPlan *pl, cudaStream_t stream, const void *W, const void *X, int x_mode, int lo_rows,
                                  int rows, int slot_rows, int N, int K, float *out, long long out_floats, GemmOut *g) {
  TcParams p;
  p.n_tok = rows; p.x_mode = x_mode; p.lo_rows = lo_rows;
  p.m_tiles = rows > TC_ROWS_MAX ? 2 : 1;
  if (rows > 2 * TC_ROWS_MAX || (p.m_tiles == 2 && (x_mode != TC_X_PLANAR || lo_rows < 2 * TC_ROWS_MAX))) return false;
  p.N = N; p.K = K; p.KB = K / TC_BK;
  p.n_tiles = (N + TC_BN - 1) / TC_BN;
  p.total_units = p.n_tiles * p.KB;
  // W stages of two panels (256-byte runs per weight row) unless the X ring needs the room
  p.wp = (x_mode == TC_X_PLANAR || p.KB < 2) ? 1 : 2;
  int grid = pl->n_sms < p.total_units ? pl->n_sms : p.total_units;
  p.upc = (p.total_units + grid - 1) / grid;
  if (p.KB % p.wp == 0) p.upc = (p.upc + p.wp - 1) / p.wp * p.wp;       // CTA ranges cover whole ring stages
  grid = (p.total_units + p.upc - 1) / p.upc;
  p.out = out;
  p.slot_stride = (long long)slot_rows * N;
  long long max_slots = (p.KB + p.upc - 1) / p.upc + 1;
  if (p.slot_stride * max_slots > out_floats) return false;
  int x_rows = x_mode == TC_X_INTERLEAVED ? 2 * rows : (x_mode == TC_X_PLANAR ? lo_rows + rows : rows);
  CUtensorMap mw, mx;
  if (!tc_map(pl, W, N, K, TC_BN, &mw) || !tc_map(pl, X, x_rows, K, 128, &mx)) return false;
  g->base = p.out; g->slot_stride = p.slot_stride; g->chunk_stride = 0; g->chunk_shift = 30; g->ld = N; g->kb = p.KB; g->upc = p.upc;
  int xstage = p.wp * (x_mode == TC_X_PLANAR ? 2 * TC_XTILE * p.m_tiles : TC_XTILE);
  p.x_stages = 2;
  int budget = pl->max_smem - 2048 - TC_STG_BYTES - p.x_stages * xstage;
  p.w_stages = budget / (p.wp * TC_WPANEL);
  if (p.w_stages > 8) p.w_stages = 8;
  if (p.w_stages < 2) return false;
  if (budget - p.w_stages * p.wp * TC_WPANEL >= xstage) p.x_stages = 3;   // room left over: a third X stage
  p.status = pl->status;
  size_t smem = (size_t)p.w_stages * p.wp * TC_WPANEL + (size_t)p.x_stages * xstage + 1024 + 512 + TC_STG_BYTES;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pl->use_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, k_gemm_tc, mw, mx, p) == cudaSuccess;
}
