// Plain CUDA-core GEMM  out[r][c] = sum_k X[r][k] W[c][k]  with fp32 accumulation.
// It serves the fp32 (toy) configuration, whose tolerances rule out tf32 tensor-core
// rounding; bf16 configurations always take the tensor-core kernel.
#pragma once
#include "common.cuh"

#define SG_BM 64
#define SG_BN 64
#define SG_BK 16

template <typename T>
__global__ void __launch_bounds__(256)
k_gemm_simt(const T *__restrict__ X, const T *__restrict__ W, float *__restrict__ out, int rows,
            int N, int K, int ldo) {
  __shared__ float As[SG_BK][SG_BM + 4];
  __shared__ float Bs[SG_BK][SG_BN + 4];
  kernel_entry(TR_k_gemm_simt);
  int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  int r0 = blockIdx.y * SG_BM, c0 = blockIdx.x * SG_BN;
  int lr = threadIdx.x >> 2, lk = (threadIdx.x & 3) * 4;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int k = k0 + lk + e;
      int ra = r0 + lr, cb = c0 + lr;
      As[lk + e][lr] = (ra < rows && k < K) ? to_f(X[(long long)ra * K + k]) : 0.f;
      Bs[lk + e][lr] = (cb < N && k < K) ? to_f(W[(long long)cb * K + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SG_BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { a[e] = As[k][ty * 4 + e]; b[e] = Bs[k][tx * 4 + e]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int r = r0 + ty * 4 + i, c = c0 + tx * 4 + j;
      if (r < rows && c < N) out[(long long)r * ldo + c] = acc[i][j];
    }
}
