// Plain CUDA-core projection Y[m][n] = sum_k X[m][k] W[n][k]; one warp per output feature.
// Bring-up and cross-check kernel.
#pragma once

#include "common.cuh"

namespace bita {

__global__ void __launch_bounds__(128) k_gemm_simple(const bf16* __restrict__ X, const bf16* __restrict__ W,
                                                     float* __restrict__ Y, int M, int N, int K, int ldy) {
  const int n = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (n >= N) return;
  const bf16* w = W + (size_t)n * K;
  for (int m = 0; m < M; ++m) {
    const bf16* x = X + (size_t)m * K;
    float acc = 0.f;
    for (int k = lane * 8; k < K; k += 256) {
      const uint4 wu = *reinterpret_cast<const uint4*>(w + k);
      const uint4 xu = *reinterpret_cast<const uint4*>(x + k);
      const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&wu);
      const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&xu);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 a = __bfloat1622float2(w2[e]), b = __bfloat1622float2(x2[e]);
        acc = fmaf(a.x, b.x, acc);
        acc = fmaf(a.y, b.y, acc);
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) Y[(size_t)m * ldy + n] = acc;
  }
}

}  // namespace bita
