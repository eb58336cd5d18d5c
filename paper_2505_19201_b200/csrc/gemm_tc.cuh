// Weight-streaming small-M GEMM for sm_100a:  out[t][c] = sum_k X[t][k] * W[c][k].
//
// The token count (<= 256 rows, hi and lo planes together) is tiny and the weight matrix is
// large, so the kernel is bound by streaming W from HBM once.  Design:
//   * swap-AB: the 128 weight rows of a tile are the MMA's M (TMEM lanes), the tokens are its
//     N (TMEM columns); one tcgen05.mma (cta_group::1, kind::f16, bf16 x bf16 -> fp32) covers
//     128 x N x 16, four per 64-wide k-block;
//   * W and X tiles arrive by TMA (cp.async.bulk.tensor.2d, 128-byte swizzle, no multicast)
//     into a ring of shared-memory stages guarded by mbarriers;
//   * persistent stream-K: the (tile, k-block) units are dealt out in equal contiguous ranges
//     to one CTA per SM, so every SM streams the same number of bytes whatever the tile count;
//     a CTA that covers part of a tile writes a partial sum to its own slot and the consumer
//     adds the (at most three) slots, in a fixed order;
//   * warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 =
//     epilogue (tcgen05.ld -> coalesced fp32 stores); two TMEM accumulators alternate so the
//     epilogue of one segment overlaps the MMAs of the next;
//   * every mbarrier wait is bounded: on expiry the kernel raises the status word and leaves.
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <map>
#include <tuple>

#include "common.cuh"

#define TC_BM 128              // weight rows per tile
#define TC_BK 64               // k elements per stage (128 bytes: one swizzle atom row)
#define TC_THREADS 192
#define TC_SPIN_LIMIT (1u << 26)

struct TcParams {
  float *out;
  long long slot_stride;       // floats
  int N, K, KB;                // output features, reduction length, k-blocks per tile
  int n_tiles, total_units, upc;
  int n_mma;                   // MMA N = token rows incl. lo plane (multiple of 16, <= 256)
  int n_tok, n_tok_pad;        // real token rows, padded rows per plane
  int lo_rows;                 // row offset of the lo plane in the X tensor map (0 = none)
  int stages, tmem_cols;
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------------------------------ kernel
// Dynamic shared memory: [stages][A tile 16 KB | B tile n_mma*128 B] (1024-byte aligned), then
// the barriers.
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t a_bytes = TC_BM * TC_BK * 2, b_bytes = (uint32_t)p.n_mma * TC_BK * 2;
  const uint32_t stage_bytes = a_bytes + b_bytes;
  uint64_t *bars = (uint64_t *)(smem + (size_t)p.stages * stage_bytes);
  uint64_t *full = bars, *empty = bars + p.stages, *acc_full = bars + 2 * p.stages, *acc_empty = acc_full + 2;
  uint32_t *tmem_base_p = (uint32_t *)(acc_empty + 2);
  volatile int *abort_flag = (volatile int *)(tmem_base_p + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long u_begin = (long long)blockIdx.x * p.upc;
  long long u_end = u_begin + p.upc;
  if (u_end > p.total_units) u_end = p.total_units;
  const bool has_work = u_begin < u_end;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full + b, 1); mbar_init(acc_empty + b, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {      // TMEM allocation by one full warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_p)), "r"((uint32_t)p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_p;

  if (has_work) {
    if (warp == 0) {
      // ------------------------------------------------------------------ TMA producer
      if (lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
        uint32_t it = 0;
        for (long long u = u_begin; u < u_end; ++u, ++it) {
          int s = it % p.stages;
          uint32_t ph = (it / p.stages) & 1;
          if (it >= (uint32_t)p.stages && !mbar_wait(empty + s, ph ^ 1)) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; break; }
          if (*abort_flag) break;
          int tile = (int)(u / p.KB), kb = (int)(u - (long long)tile * p.KB);
          uint8_t *sa = smem + (size_t)s * stage_bytes, *sb = sa + a_bytes;
          mbar_expect_tx(full + s, stage_bytes);
          tma_load_2d(sa, &map_w, full + s, kb * TC_BK, tile * TC_BM, pol_w);
          tma_load_2d(sb, &map_x, full + s, kb * TC_BK, 0, pol_x);
          if (p.lo_rows) tma_load_2d(sb + (size_t)p.n_tok_pad * TC_BK * 2, &map_x, full + s, kb * TC_BK, p.lo_rows, pol_x);
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------------ MMA issuer
      if (lane == 0) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_mma >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
        uint32_t it = 0, seg = 0;
        long long u = u_begin;
        bool ok = true;
        while (u < u_end && ok) {
          int tile = (int)(u / p.KB);
          long long seg_end = (long long)(tile + 1) * p.KB;
          if (seg_end > u_end) seg_end = u_end;
          int buf = seg & 1;
          if (seg >= 2 && !mbar_wait(acc_empty + buf, ((seg >> 1) & 1) ^ 1)) { ok = false; break; }
          tc_fence_after();
          uint32_t d_addr = tmem_base + (uint32_t)buf * (uint32_t)p.n_mma;
          bool first = true;
          for (; u < seg_end; ++u, ++it) {
            int s = it % p.stages;
            if (!mbar_wait(full + s, (it / p.stages) & 1)) { ok = false; break; }
            tc_fence_after();
            uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
            uint64_t ad = smem_desc(sa), bd = smem_desc(sb);
#pragma unroll
            for (int k = 0; k < TC_BK / 16; ++k) {
              mma_bf16(d_addr, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), idesc, (first && k == 0) ? 0u : 1u);
            }
            first = false;
            mma_commit(empty + s);            // frees the stage once these MMAs have read it
          }
          if (!ok) break;
          mma_commit(acc_full + buf);         // accumulator complete
          ++seg;
        }
        if (!ok) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; }
      }
    } else {
      // ------------------------------------------------------------------ epilogue warps
      const int q = warp & 3;                 // TMEM lane quarter this warp may read
      uint32_t seg = 0;
      long long u = u_begin;
      while (u < u_end) {
        int tile = (int)(u / p.KB);
        long long seg_end = (long long)(tile + 1) * p.KB;
        if (seg_end > u_end) seg_end = u_end;
        int buf = seg & 1;
        bool ok = mbar_wait(acc_full + buf, (seg >> 1) & 1);
        if (!ok || *abort_flag) { if (lane == 0) { atomicMax(p.status, DREAM_DEV_TIMEOUT); *abort_flag = 1; } break; }
        tc_fence_after();
        int first_cta = (int)(((long long)tile * p.KB) / p.upc);
        int slot = (int)blockIdx.x - first_cta;
        int c = tile * TC_BM + q * 32 + lane;
        float *dst = p.out + (long long)slot * p.slot_stride + c;
        uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * (uint32_t)p.n_mma;
        for (int col0 = 0; col0 < p.n_mma; col0 += 16) {
          uint32_t r[16];
          tmem_ld16(taddr + (uint32_t)col0, r);
          tmem_ld_wait();
          if (c < p.N) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              int col = col0 + j;
              int t = col < p.n_tok_pad ? col : col - p.n_tok_pad;
              if (t < p.n_tok) dst[(long long)col * p.N] = __uint_as_float(r[j]);
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
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ host side

struct GemmTcPlan {
  PFN_cuTensorMapEncodeTiled_v12000 encode;
  int n_sms;
  int max_smem;
  int *status;
  std::map<std::tuple<const void *, int, int, int>, CUtensorMap> maps;
};

static inline const char *gemm_tc_plan_init(GemmTcPlan *pl, int *status) {
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
  return nullptr;
}

static inline bool gemm_tc_supported(int rows_total, int N, int K) {
  return rows_total >= 16 && rows_total <= 256 && rows_total % 16 == 0 && K % TC_BK == 0 && K >= TC_BK && N % 8 == 0 && N >= 8;
}

// bf16 row-major [rows][K] matrix, box = 64 x box_rows, 128-byte swizzle.
static inline const CUtensorMap *tc_map(GemmTcPlan *pl, const void *ptr, int rows, int K, int box_rows) {
  auto key = std::make_tuple(ptr, rows, K, box_rows);
  auto it = pl->maps.find(key);
  if (it != pl->maps.end()) return &it->second;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {TC_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = pl->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return nullptr;
  if (pl->maps.size() > 4096) pl->maps.clear();
  return &(pl->maps[key] = m);
}

// Enqueue one GEMM.  X holds `rows` token rows (hi plane) and, when lo_delta != 0, their
// low-order parts lo_delta elements further on.  Returns false if a tensor map could not be made.
static inline bool gemm_tc_launch(GemmTcPlan *pl, cudaStream_t stream, const void *W, const void *X, long long lo_delta,
                                  int rows, int N, int K, float *out, long long out_floats, GemmOut *g) {
  TcParams p;
  p.n_tok = rows;
  p.n_tok_pad = (rows + 15) & ~15;
  p.n_mma = p.n_tok_pad * (lo_delta ? 2 : 1);
  p.lo_rows = lo_delta ? (int)(lo_delta / K) : 0;
  p.N = N; p.K = K; p.KB = K / TC_BK;
  p.n_tiles = (N + TC_BM - 1) / TC_BM;
  p.total_units = p.n_tiles * p.KB;
  int grid = pl->n_sms < p.total_units ? pl->n_sms : p.total_units;
  p.upc = (p.total_units + grid - 1) / grid;
  grid = (p.total_units + p.upc - 1) / p.upc;
  int stage_bytes = TC_BM * TC_BK * 2 + p.n_mma * TC_BK * 2;
  int budget = pl->max_smem - 2048;
  p.stages = budget / stage_bytes;
  if (p.stages > 12) p.stages = 12;
  if (p.stages < 2) return false;
  int cols = 2 * p.n_mma;
  p.tmem_cols = 32;
  while (p.tmem_cols < cols) p.tmem_cols <<= 1;
  p.out = out;
  p.slot_stride = (long long)p.n_mma * N;
  long long max_slots = (p.KB + p.upc - 1) / p.upc + 1;
  if (p.slot_stride * max_slots > out_floats) return false;
  p.status = pl->status;
  int x_rows = p.lo_rows + p.n_tok_pad;
  const CUtensorMap *mw = tc_map(pl, W, N, K, TC_BM);
  const CUtensorMap *mx = tc_map(pl, X, x_rows, K, p.n_tok_pad);
  if (!mw || !mx) return false;
  size_t smem = (size_t)p.stages * stage_bytes + 1024 + 256;
  k_gemm_tc<<<grid, TC_THREADS, smem, stream>>>(*mw, *mx, p);
  g->base = out; g->slot_stride = p.slot_stride; g->ld = N; g->kb = p.KB; g->upc = p.upc;
  g->lo_off = lo_delta ? p.n_tok_pad : 0;
  return true;
}
