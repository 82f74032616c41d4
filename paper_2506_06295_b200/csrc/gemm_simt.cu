// C[M,N] (fp32) = A[M,K] * W[N,K]^T on the plain fp32 ALUs.
//
// This is the GEMM of the fp32 mode (the tiny configuration asks for 1e-4
// relative error, which TF32 tensor cores do not give) and the independent
// cross-check for the tensor-core kernel in tests.  64x64 output tile, 16x16
// threads, 4x4 outputs per thread, K staged through shared memory 16 at a time.
#include "internal.h"

namespace dllm {

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ W,
                                                        float* __restrict__ C, int M, int N, int K) {
  pdl_wait();
  pdl_trigger();
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += BK) {
    // 64 rows x 16 k per operand = 1024 elements, 4 per thread
    for (int e = threadIdx.x; e < BM * BK; e += 256) {
      const int r = e / BK, kk = e - r * BK;
      const int gm = m0 + r, gn = n0 + r, gk = k0 + kk;
      As[kk][r] = (gm < M && gk < K) ? to_f32<T>(A[(size_t)gm * K + gk]) : 0.f;
      Ws[kk][r] = (gn < N && gk < K) ? to_f32<T>(W[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = Ws[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn < N) C[(size_t)gm * N + gn] = acc[i][j];
    }
  }
}

void launch_gemm_simt(const Launch& L, int dtype, const void* A, const void* W, float* C, int M, int N, int K) {
  if (M <= 0 || N <= 0) return;
  dim3 grid((N + 63) / 64, (M + 63) / 64);
  if (dtype == 0)
    launch_k(L, gemm_simt_kernel<float>, dim3(grid), dim3(256), 0, (const float*)A, (const float*)W, C, M, N, K);
  else
    launch_k(L, gemm_simt_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, (const __nv_bfloat16*)A, (const __nv_bfloat16*)W, C, M, N, K);
  L.count();
}

}  // namespace dllm

DLLM_TIMELINE_HOOKS(gemm_simt)
