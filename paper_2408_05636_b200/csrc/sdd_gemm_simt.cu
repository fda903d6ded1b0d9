// CUDA-core GEMM  C[M, N] = A[M, K] * W[N, K]^T  with fused epilogues.
// This is the contraction of the fp32 configuration (fp32 storage and accumulation, where tensor
// cores have no fp32 operand type) and a slow cross-check of the bf16 tensor-core GEMM.
#include "sdd_kernels.h"

namespace sdd {

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16, SG_THREADS = 256;

template <typename T>
__global__ void __launch_bounds__(SG_THREADS)
gemm_simt_kernel(const T* __restrict__ A, int lda, const T* __restrict__ W, const float* __restrict__ bias, int M, int N,
                 int K, int epi, void* __restrict__ out, int ldc, const int* __restrict__ skip) {
  pdl_launch_dependents();
  pdl_wait();
  if (skip != nullptr && *skip) return;
  __shared__ float As[SG_BK][SG_BM + 4];
  __shared__ float Ws[SG_BK][SG_BN + 4];
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;   // 16 x 16 threads, 4 x 4 outputs each
  const int lr = threadIdx.x >> 2, lk = (threadIdx.x & 3) * 4;  // loader: 64 rows x 4 k-quads
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int k = k0 + lk + q;
      const int am = m0 + lr, wn = n0 + lr;
      As[lk + q][lr] = (am < M && k < K) ? to_f32(A[(long long)am * lda + k]) : 0.f;
      Ws[lk + q][lr] = (wn < N && k < K) ? to_f32(W[(long long)wn * K + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SG_BK; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j] + (bias != nullptr ? bias[n] : 0.f);
      const long long o = (long long)m * ldc + n;
      if (epi == EPI_STORE) reinterpret_cast<T*>(out)[o] = from_f32<T>(v);
      else if (epi == EPI_GELU) reinterpret_cast<T*>(out)[o] = from_f32<T>(gelu_tanh(v));
      else if (epi == EPI_RESIDUAL) reinterpret_cast<float*>(out)[o] += v;
      else reinterpret_cast<float*>(out)[o] = v;
    }
  }
}

template <typename T>
cudaError_t launch_gemm_simt(const T* A, int lda, const T* W, const float* bias, int M, int N, int K, int epi, void* out,
                             int ldc, cudaStream_t st, const int* skip) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  dim3 grid((N + SG_BN - 1) / SG_BN, (M + SG_BM - 1) / SG_BM);
  launch_k(gemm_simt_kernel<T>, dim3(grid), dim3(SG_THREADS), 0, st, A, lda, W, bias, M, N, K, epi, out, ldc, skip);
  return cudaGetLastError();
}

template cudaError_t launch_gemm_simt<float>(const float*, int, const float*, const float*, int, int, int, int, void*, int,
                                             cudaStream_t, const int*);
template cudaError_t launch_gemm_simt<__nv_bfloat16>(const __nv_bfloat16*, int, const __nv_bfloat16*, const float*, int,
                                                     int, int, int, void*, int, cudaStream_t, const int*);

}  // namespace sdd
