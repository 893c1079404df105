// Recurrent step of the two further token-mixer variants of the Architecture section, as stand-alone kernels
// on normed inputs z[R, d] (fp32): linearly combined heads (each head owns a row-repeat and a column-repeat
// matrix and outputs a linear combination of the two products: Eq. 2 and Eq. 3 side by side, twice the cache)
// and non-unitary kernels (Eq. 11: k column-repeat filters, filter i reading the hidden channels shifted by i,
// zero beyond the last channel; k times the cache). Both are streams over the cache: HBM-bound.
#pragma once

#include "common.cuh"

namespace srm {

struct CombinedParams {
  int64_t R;
  int d, h, t, n_ctx;
  const float* z;                 // [R, d]
  float *S_row, *S_col;           // [R, d] each, in/out
  const float *alpha_row, *alpha_col;   // [h, n_ctx]
  const float* beta;              // [n_ctx, d]
  const float *lam_row, *lam_col; // [h]
  const float* w;                 // [h, 2]: weight of the row-repeat and of the column-repeat product
  float* y;                       // [R, d]
};

// Bytes per row: d * 4 * (z + 2 caches read + 2 caches written + y) = 24 d.
//   y    = w_row (alpha_row[t] z + S_row) + w_col alpha_col[t] (z + S_col) + beta_t
//   S_row <- lam_row (S_row + alpha_row[t] z);  S_col <- lam_col (S_col + z)
constexpr int kVariantThreads = 256;
__global__ void __launch_bounds__(kVariantThreads) combined_step_kernel(const CombinedParams p) {
  pdl_trigger();
  pdl_wait();
  const int q = p.d >> 2, dh = p.d / p.h;
  const int64_t n4 = p.R * q;
  for (int64_t idx = (int64_t)blockIdx.x * kVariantThreads + threadIdx.x; idx < n4; idx += (int64_t)gridDim.x * kVariantThreads) {
    const int64_t row = idx / q;
    const int c = (int)(idx - row * q) << 2;
    const int g = c / dh;
    const float ar = __ldg(p.alpha_row + (int64_t)g * p.n_ctx + p.t), ac = __ldg(p.alpha_col + (int64_t)g * p.n_ctx + p.t);
    const float lr = __ldg(p.lam_row + g), lc = __ldg(p.lam_col + g);
    const float wr = __ldg(p.w + 2 * g), wc = __ldg(p.w + 2 * g + 1) * ac;
    const int64_t o = row * p.d + c;
    const float4 z = ld4(p.z + o), sr = ld4(p.S_row + o), sc = ld4(p.S_col + o);
    const float4 bt = ldg4(p.beta + (int64_t)p.t * p.d + c);
    const float4 u = make_float4(ar * z.x, ar * z.y, ar * z.z, ar * z.w);
    const float4 v = make_float4(z.x + sc.x, z.y + sc.y, z.z + sc.z, z.w + sc.w);
    float4 y;
    y.x = fmaf(wr, u.x + sr.x, fmaf(wc, v.x, bt.x)); y.y = fmaf(wr, u.y + sr.y, fmaf(wc, v.y, bt.y));
    y.z = fmaf(wr, u.z + sr.z, fmaf(wc, v.z, bt.z)); y.w = fmaf(wr, u.w + sr.w, fmaf(wc, v.w, bt.w));
    st4(p.y + o, y);
    st4(p.S_row + o, make_float4(lr * (sr.x + u.x), lr * (sr.y + u.y), lr * (sr.z + u.z), lr * (sr.w + u.w)));
    st4(p.S_col + o, make_float4(lc * v.x, lc * v.y, lc * v.z, lc * v.w));
  }
}

struct KernelMixParams {
  int64_t R;
  int d, k, t, n_ctx;
  const float* z;        // [R, d]
  float* P;              // [k, R, d] in/out: the column-repeat sum term of every filter
  const float* alpha;    // [k, n_ctx]
  const float* beta;     // [n_ctx, d]
  const float* lam;      // [k]
  float* y;              // [R, d]
};
constexpr int kKernelMixMaxK = 16;
inline size_t kernel_mix_smem(int d, int k) { return (size_t)k * d * 4 + 2 * kKernelMixMaxK * 4; }

// One CTA walks rows. Per row: v_i = z + P_i for the k filters (written to shared memory, lam_i v_i back to the
// cache), then y[c] = beta_t[c] + sum_i alpha_i[t] v_i[c + i] with the terms past the last channel dropped
// (the zero padding of Eq. 11). Bytes per row: d * 4 * (2 k + 2).
__global__ void __launch_bounds__(kVariantThreads) kernel_mix_step_kernel(const KernelMixParams p) {
  pdl_trigger();
  extern __shared__ __align__(16) float vs[];           // [k][d], then alpha_i[t], lam_i
  const int d = p.d, k = p.k;
  float* a_s = vs + (size_t)k * d;
  float* l_s = a_s + kKernelMixMaxK;
  if (threadIdx.x < k) {
    a_s[threadIdx.x] = __ldg(p.alpha + (int64_t)threadIdx.x * p.n_ctx + p.t);
    l_s[threadIdx.x] = __ldg(p.lam + threadIdx.x);
  }
  __syncthreads();
  pdl_wait();
  const float* bt = p.beta + (int64_t)p.t * d;
  const int64_t plane = p.R * (int64_t)d;
  for (int64_t row = blockIdx.x; row < p.R; row += gridDim.x) {
    for (int e = threadIdx.x * 4; e < d; e += kVariantThreads * 4) {
      const float4 z = ld4(p.z + row * d + e);
      float* P0 = p.P + row * d + e;
      for (int i0 = 0; i0 < k; i0 += 4) {          // four filters' loads in flight before the first store
        float4 s[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (i0 + u < k) s[u] = ld4(P0 + (int64_t)(i0 + u) * plane);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (i0 + u < k) {
            const float4 v = make_float4(z.x + s[u].x, z.y + s[u].y, z.z + s[u].z, z.w + s[u].w);
            st4(vs + (size_t)(i0 + u) * d + e, v);
            const float l = l_s[i0 + u];
            st4(P0 + (int64_t)(i0 + u) * plane, make_float4(l * v.x, l * v.y, l * v.z, l * v.w));
          }
        }
      }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < d; c += kVariantThreads) {
      float acc = __ldg(bt + c);
      const int kk = d - c < k ? d - c : k;
      for (int i = 0; i < kk; ++i) acc = fmaf(a_s[i], vs[(size_t)i * d + c + i], acc);
      p.y[row * d + c] = acc;
    }
    __syncthreads();
  }
}

}  // namespace srm
