// Shared device helpers of the DREAM hot path: element conversion, deterministic block
// reductions, the split-output descriptor every GEMM consumer reads through.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

#define DREAM_MAX_BATCH 8          // sequences one call may list

#define DREAM_DEV_OK 0
#define DREAM_DEV_TIMEOUT 1
#define DREAM_DEV_BAD_INDEX 2

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// Programmatic dependent launch: a kernel may start while its predecessor in the stream is still
// running; pdl_wait() blocks until the predecessor has completed and its writes are visible, and
// pdl_trigger() lets the successor start early.  Every kernel of the library calls pdl_wait()
// before it touches memory another kernel writes (weights never change and may be read earlier).
// Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Optional timeline of a stream: when a trace buffer is installed (dream_trace), thread 0 of block
// 0 of every kernel appends (kernel id, %globaltimer) right after its grid dependency resolved,
// i.e. when its predecessor has completed.  Differences between consecutive entries are the
// critical-path time of each kernel as it runs in the stream, overlap included.  Layout of the
// buffer: word 0 = entries written, word 1 = capacity, then pairs (id, nanoseconds).
__device__ unsigned long long *g_dream_trace;
enum {
  TR_none = 0,
  TR_k_embed,
  TR_k_build_prompt,
  TR_k_resid_norm,
  TR_k_qkv_post_target,
  TR_k_qkv_post_draft,
  TR_k_gemm_to_q,
  TR_k_mem_append,
  TR_k_silu_mul,
  TR_k_resid_add,
  TR_k_gather_rows,
  TR_k_topk_lse,
  TR_k_attn_prefill,
  TR_k_entropy_mean,
  TR_k_colsum,
  TR_k_attn_tree,
  TR_k_attn_draft,
  TR_k_attn_tc,
  TR_k_attn_combine,
  TR_k_draft_begin,
  TR_k_tree_expand,
  TR_k_tree_finalize,
  TR_k_verify_setup,
  TR_k_accept,
  TR_k_compact_kv,
  TR_k_accept_rows,
  TR_k_select_tap,
  TR_k_select_visual,
  TR_k_ctx_rows,
  TR_k_gemm_simt,
  TR_k_iota_rows,
  TR_k_set_seq,
  TR_k_set_int,
  TR_k_first_token,
  TR_k_argmax_out,
  TR_k_copy_f32,
  TR_k_split_rows,
  TR_k_gemm_collect,
  TR_k_gemm_tc,
  TR_count
};
#define DREAM_TRACE_NAMES {"none", "k_embed", "k_build_prompt", "k_resid_norm", "k_qkv_post_target", "k_qkv_post_draft", "k_gemm_to_q", "k_mem_append", "k_silu_mul", "k_resid_add", "k_gather_rows", "k_topk_lse", "k_attn_prefill", "k_entropy_mean", "k_colsum", "k_attn_tree", "k_attn_draft", "k_attn_tc", "k_attn_combine", "k_draft_begin", "k_tree_expand", "k_tree_finalize", "k_verify_setup", "k_accept", "k_compact_kv", "k_accept_rows", "k_select_tap", "k_select_visual", "k_ctx_rows", "k_gemm_simt", "k_iota_rows", "k_set_seq", "k_set_int", "k_first_token", "k_argmax_out", "k_copy_f32", "k_split_rows", "k_gemm_collect", "k_gemm_tc"}
__device__ __forceinline__ void trace_stamp(int id) {
  unsigned long long *tr = g_dream_trace;
  if (tr) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    unsigned long long i = atomicAdd(tr, 1ull);
    if (i < tr[1]) { tr[2 + 2 * i] = (unsigned long long)id; tr[3 + 2 * i] = t; }
  }
}
// Entry of every kernel of the library: let the successor start, wait for the predecessor.
__device__ __forceinline__ void kernel_entry(int id) {
  pdl_trigger();
  pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) trace_stamp(id);
}

// The same, for a kernel that wants its successor to start only when it is about to finish (a
// successor that fills the SMs' shared memory would otherwise crowd it out): it calls
// pdl_trigger() itself, late.
__device__ __forceinline__ void kernel_entry_late(int id) {
  pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) trace_stamp(id);
}

// Weights never change, so a kernel that leaves HBM idle can pull the next GEMM's weights into the
// 126 MB L2 ahead of time, before its own grid dependency resolves.  Every CTA requests an equal
// slice with bulk L2 prefetches issued by one thread.
struct L2Prefetch {
  const char *ptr;               // 128-byte aligned; null = nothing to fetch
  unsigned long long bytes;
};
__device__ __forceinline__ void l2_prefetch_slice(const L2Prefetch &pf, unsigned cta, unsigned n_cta) {
  if (!pf.ptr || threadIdx.x != 0) return;
  unsigned long long per = ((pf.bytes + n_cta - 1) / n_cta + 127ull) & ~127ull;
  unsigned long long lo = per * cta, hi = lo + per < pf.bytes ? lo + per : pf.bytes;
  for (unsigned long long o = lo; o < hi; o += 32768ull) {
    unsigned sz = (unsigned)((hi - o < 32768ull ? hi - o : 32768ull) & ~15ull);
    if (sz) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(pf.ptr + o), "r"(sz) : "memory");
  }
}

// A bf16 GEMM input row is stored as two bf16 rows, hi = bf16(v) and lo = bf16(v - hi), so the
// tensor cores see the activation to ~16 mantissa bits while the weights stream once.  fp32
// inputs have no lo part.  XLayout says where the rows of such a buffer live: token t starts at
// element t * row_stride, and its lo part lo_delta elements further on (0 = no lo part).
struct XLayout {
  long long row_stride;
  long long lo_delta;
};
template <typename T> __device__ __forceinline__ void store_split(T *p, long long lo_delta, float v);
template <> __device__ __forceinline__ void store_split<float>(float *p, long long, float v) { *p = v; }
template <> __device__ __forceinline__ void store_split<bf16>(bf16 *p, long long lo_delta, float v) {
  bf16 hi = __float2bfloat16_rn(v);
  *p = hi;
  if (lo_delta) p[lo_delta] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Output of a GEMM: rows are cut into chunks of (1 << chunk_shift) rows, one launch each,
// chunk_stride floats apart.  Inside a chunk the stream-K tensor-core kernel leaves up to
// ceil(kb / upc) + 1 partial sums per 256-column tile, stacked in slots of slot_stride floats; the
// SIMT kernel leaves one (upc == 0).
struct GemmOut {
  const float *base;
  long long slot_stride;   // floats between consecutive slots
  long long chunk_stride;  // floats between consecutive row chunks
  int chunk_shift;         // log2 of the rows per chunk
  int ld;                  // floats between consecutive rows (tokens)
  int kb;                  // k-panels per tile
  int upc;                 // work units (tile, k-panel) per CTA; 0 = single slot
};

__device__ __forceinline__ float gemm_val(const GemmOut &g, int r, int c) {
  int ch = r >> g.chunk_shift;
  const float *p = g.base + (long long)ch * g.chunk_stride + (long long)(r - (ch << g.chunk_shift)) * g.ld + c;
  float s = *p;
  if (g.upc) {
    unsigned u0 = (unsigned)(c >> 8) * (unsigned)g.kb;
    int extra = (int)((u0 + (unsigned)g.kb - 1u) / (unsigned)g.upc) - (int)(u0 / (unsigned)g.upc);
    for (int i = 1; i <= extra; ++i) s += p[(long long)i * g.slot_stride];
  }
  return s;
}

// Four consecutive columns c..c+3 (c a multiple of 4: they share a tile, hence a slot count).
// The slots are added in slot order, but fetched four at a time so that a value made of many
// partial sums costs a few memory round trips instead of one per slot.
__device__ __forceinline__ void add4(float4 &s, const float4 &t) { s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w; }
__device__ __forceinline__ int gemm_extra_slots(const GemmOut &g, int c) {
  if (!g.upc) return 0;
  unsigned u0 = (unsigned)(c >> 8) * (unsigned)g.kb;
  return (int)((u0 + (unsigned)g.kb - 1u) / (unsigned)g.upc) - (int)(u0 / (unsigned)g.upc);
}
__device__ __forceinline__ float4 gemm_val4(const GemmOut &g, int r, int c) {
  int ch = r >> g.chunk_shift;
  const float4 *p = reinterpret_cast<const float4 *>(g.base + (long long)ch * g.chunk_stride +
                                                     (long long)(r - (ch << g.chunk_shift)) * g.ld + c);
  float4 s = *p;
  const int extra = gemm_extra_slots(g, c);
  const long long st4 = g.slot_stride >> 2;
  int i = 1;
  for (; i + 3 <= extra; i += 4) {
    float4 t0 = p[(long long)i * st4], t1 = p[(long long)(i + 1) * st4], t2 = p[(long long)(i + 2) * st4], t3 = p[(long long)(i + 3) * st4];
    add4(s, t0); add4(s, t1); add4(s, t2); add4(s, t3);
  }
  if (i + 1 <= extra) {
    float4 t0 = p[(long long)i * st4], t1 = p[(long long)(i + 1) * st4];
    add4(s, t0); add4(s, t1);
    i += 2;
  }
  if (i <= extra) { float4 t0 = p[(long long)i * st4]; add4(s, t0); }
  return s;
}

// The same with up to MAXS extra slots fetched per round trip (more registers; for consumers that
// read values made of many partial sums, such as the outputs of the narrow projections).
template <int MAXS>
__device__ __forceinline__ float4 gemm_val4_wide(const GemmOut &g, int r, int c) {
  int ch = r >> g.chunk_shift;
  const float4 *p = reinterpret_cast<const float4 *>(g.base + (long long)ch * g.chunk_stride +
                                                     (long long)(r - (ch << g.chunk_shift)) * g.ld + c);
  float4 s = *p;
  const int extra = gemm_extra_slots(g, c);
  const long long st4 = g.slot_stride >> 2;
  for (int i = 1; i <= extra; i += MAXS) {
    float4 t[MAXS];
#pragma unroll
    for (int k = 0; k < MAXS; ++k) t[k] = i + k <= extra ? p[(long long)(i + k) * st4] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int k = 0; k < MAXS; ++k) add4(s, t[k]);
  }
  return s;
}

// Four consecutive elements of a GEMM input row, high (and low) parts, as 8-byte stores.
template <typename T> __device__ __forceinline__ void store_split4(T *p, long long lo_delta, float4 v);
template <> __device__ __forceinline__ void store_split4<float>(float *p, long long, float4 v) {
  *reinterpret_cast<float4 *>(p) = v;
}
template <> __device__ __forceinline__ void store_split4<bf16>(bf16 *p, long long lo_delta, float4 v) {
  __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
  uint2 hv = make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
  *reinterpret_cast<uint2 *>(p) = hv;
  if (lo_delta) {
    float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
    __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - f0.x, v.y - f0.y), l1 = __floats2bfloat162_rn(v.z - f1.x, v.w - f1.y);
    *reinterpret_cast<uint2 *>(p + lo_delta) = make_uint2(*reinterpret_cast<uint32_t *>(&l0), *reinterpret_cast<uint32_t *>(&l1));
  }
}
__device__ __forceinline__ float4 ld_f4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 ld_f4(const bf16 *p) {
  uint2 u = *reinterpret_cast<const uint2 *>(p);
  float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162 *>(&u.x)), b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162 *>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}

// Query rows between the QKV post-processing and the attention kernels: one block of hd
// values per (row, head): fp32 (fp32 configurations), or hd high parts then hd low parts in bf16
// (bf16 configurations: what the tensor-core attention copies straight into shared memory).
// Four bytes per element either way.  rh = row * H + head.
__device__ __forceinline__ void q_store4(void *qbuf, int split, long long rh, int hd, int i, float4 v) {
  if (split) store_split4<bf16>((bf16 *)qbuf + rh * 2 * hd + i, hd, v);
  else *reinterpret_cast<float4 *>((float *)qbuf + rh * hd + i) = v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Sum over a block of up to 1024 threads, same value returned to every thread; the order
// of additions is fixed, so results are reproducible run to run.
__device__ __forceinline__ float block_sum(float v, float *sh /* >= 33 floats */) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  if (w == 0) {
    float t = lane < nw ? sh[lane] : 0.f;
    t = warp_sum(t);
    if (lane == 0) sh[32] = t;
  }
  __syncthreads();
  return sh[32];
}

// (value, index) ordering used by every top-k / argmax: larger value first, then lower index.
__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}
