// Plain SIMT projection D[M,N] = A[M,K] * W[N,K]^T with fp32 FMA accumulation in K order.
// Used for the fp32 configuration (where TF32/bf16 tensor cores would break the 1e-4 bound)
// and as an on-device cross-check of the tensor-core kernel. Not performance-critical.
#pragma once

#include "common.cuh"

namespace srm {

enum GemmEpilogue {
  kEpiBiasGelu = 0,       // out = gelu(D + bias) in the activation type
  kEpiBiasResidual = 1,   // out += D + bias (fp32)
  kEpiPlain = 2,          // out = D (fp32)
  kEpiArgmax = 3,         // tensor-core kernel only: per-row (max, lowest column) of every 64-column slice of D
  kEpiCollect = 4         // tensor-core kernel only: per row, every element of D at or above the row's threshold is
                          // appended to the row's candidate list (top-k selection without writing D)
};

constexpr int kSimtBM = 64, kSimtBN = 64, kSimtBK = 16;

template <typename T, int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ W, const float* __restrict__ bias,
                 void* __restrict__ out, int64_t M, int64_t N, int64_t K) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sA[kSimtBK][kSimtBM + 4];
  __shared__ float sW[kSimtBK][kSimtBN + 4];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * kSimtBM, n0 = (int64_t)blockIdx.x * kSimtBN;
  float acc[4][4] = {};
  // loader mapping: 256 threads fetch 64 rows x 16 k, one 4-wide vector each
  const int lr = threadIdx.x >> 2, lk = (threadIdx.x & 3) * 4;
  for (int64_t k0 = 0; k0 < K; k0 += kSimtBK) {
    float4 va = make_float4(0.f, 0.f, 0.f, 0.f), vw = va;
    if (m0 + lr < M) va = ld4(A + (m0 + lr) * K + k0 + lk);
    if (n0 + lr < N) vw = ld4(W + (n0 + lr) * K + k0 + lk);
    sA[lk + 0][lr] = va.x; sA[lk + 1][lr] = va.y; sA[lk + 2][lr] = va.z; sA[lk + 3][lr] = va.w;
    sW[lk + 0][lr] = vw.x; sW[lk + 1][lr] = vw.y; sW[lk + 2][lr] = vw.z; sW[lk + 3][lr] = vw.w;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kSimtBK; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sA[k][ty * 4 + i]; w[i] = sW[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j];
      if (EPI == kEpiBiasGelu) {
        reinterpret_cast<T*>(out)[m * N + n] = from_float<T>(gelu_erf(v + bias[n]));
      } else if (EPI == kEpiBiasResidual) {
        float* o = reinterpret_cast<float*>(out) + m * N + n;
        *o = *o + (bias != nullptr ? v + bias[n] : v);
      } else {
        reinterpret_cast<float*>(out)[m * N + n] = v;
      }
    }
  }
}

}  // namespace srm
