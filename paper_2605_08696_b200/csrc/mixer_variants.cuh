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

// ---- the same two variants over whole sequences (the prefill form, through the recurrence) -----------------
// Z[Bp, n, d] holds n consecutive positions t0 .. t0 + n - 1 of Bp samples; the caches enter as the sum terms
// for position t0 (zeros for a fresh prompt) and leave as the sum terms for position t0 + n. The result equals
// the product with the explicit n x n matrices of Eq. 1 / Eq. 3 (and Eq. 11) up to rounding order.

struct CombinedScanParams {
  int64_t Bp;
  int n, t0, d, h, n_ctx;
  const float* Z;                 // [Bp, n, d]
  float *S_row, *S_col;           // [Bp, d] in/out
  const float *alpha_row, *alpha_col, *beta, *lam_row, *lam_col, *w;
  float* Y;                       // [Bp, n, d]
};

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int kCombinedRing = 8;           // positions of input in flight per thread
// One thread owns four channels of one sample and walks the positions with both sum terms in registers; its
// inputs of the next seven positions are on their way into a private ring in shared memory (16-byte asynchronous
// copies; they do not depend on the recurrence). 8 d bytes per position.
__global__ void __launch_bounds__(kVariantThreads) combined_scan_kernel(const CombinedScanParams p) {
  pdl_trigger();
  __shared__ __align__(16) float rings[kVariantThreads * kCombinedRing * 4];
  float* ring = rings + threadIdx.x * 4;          // this thread's slots, kVariantThreads * 4 floats apart (no bank conflicts)
  pdl_wait();
  const int q = p.d >> 2, dh = p.d / p.h;
  const int64_t n4 = p.Bp * q;
  for (int64_t idx = (int64_t)blockIdx.x * kVariantThreads + threadIdx.x; idx < n4; idx += (int64_t)gridDim.x * kVariantThreads) {
    const int64_t b = idx / q;
    const int c = (int)(idx - b * q) << 2;
    const int g = c / dh;
    const float lr = __ldg(p.lam_row + g), lc = __ldg(p.lam_col + g);
    const float wr = __ldg(p.w + 2 * g), wc0 = __ldg(p.w + 2 * g + 1);
    const float* ar_g = p.alpha_row + (int64_t)g * p.n_ctx + p.t0;
    const float* ac_g = p.alpha_col + (int64_t)g * p.n_ctx + p.t0;
    const float* bt = p.beta + (int64_t)p.t0 * p.d + c;
    const float* zp = p.Z + b * p.n * (int64_t)p.d + c;
    float* yp = p.Y + b * p.n * (int64_t)p.d + c;
    float4 sr = ld4(p.S_row + b * p.d + c), sc = ld4(p.S_col + b * p.d + c);
    auto issue = [&](int jj) {                 // one group per position, empty past the end
      if (jj < p.n) cp_async16(ring + (jj % kCombinedRing) * (kVariantThreads * 4), zp + (int64_t)jj * p.d);
      cp_async_commit();
    };
#pragma unroll
    for (int jj = 0; jj < kCombinedRing - 1; ++jj) issue(jj);
    for (int j = 0; j < p.n; ++j) {
      issue(j + kCombinedRing - 1);            // into the slot read one position ago
      cp_async_wait<kCombinedRing - 1>();
      const float4 z = ld4(ring + (j % kCombinedRing) * (kVariantThreads * 4));
      const float ar = __ldg(ar_g + j), wc = wc0 * __ldg(ac_g + j);
      const float4 b4 = ldg4(bt + (int64_t)j * p.d);
      const float4 uu = make_float4(ar * z.x, ar * z.y, ar * z.z, ar * z.w);
      const float4 v = make_float4(z.x + sc.x, z.y + sc.y, z.z + sc.z, z.w + sc.w);
      float4 y;
      y.x = fmaf(wr, uu.x + sr.x, fmaf(wc, v.x, b4.x)); y.y = fmaf(wr, uu.y + sr.y, fmaf(wc, v.y, b4.y));
      y.z = fmaf(wr, uu.z + sr.z, fmaf(wc, v.z, b4.z)); y.w = fmaf(wr, uu.w + sr.w, fmaf(wc, v.w, b4.w));
      st4(yp + (int64_t)j * p.d, y);
      sr = make_float4(lr * (sr.x + uu.x), lr * (sr.y + uu.y), lr * (sr.z + uu.z), lr * (sr.w + uu.w));
      sc = make_float4(lc * v.x, lc * v.y, lc * v.z, lc * v.w);
    }
    cp_async_wait<0>();
    st4(p.S_row + b * p.d + c, sr);
    st4(p.S_col + b * p.d + c, sc);
  }
}

struct KernelScanParams {
  int64_t Bp;
  int n, t0, d, k, n_ctx;
  const float* Z;        // [Bp, n, d]
  float* P;              // [k, Bp, d] in/out
  const float *alpha, *beta, *lam;
  float* Y;              // [Bp, n, d]
};
constexpr int kScanRing = 4;               // positions of input and beta rows in flight per CTA
inline size_t kernel_scan_smem(int d, int k) { return (2 * (size_t)k + 2 * kScanRing) * d * 4 + 2 * kKernelMixMaxK * 4; }

// One CTA owns a sample: the k sum terms live in shared memory for the whole sequence (each element touched by
// one thread only), the k vectors z + P_i of the current position in a second slab that the shifted reads of
// Eq. 11 take after a barrier. The input row and the beta row of the next kScanRing - 1 positions are on their
// way into a shared-memory ring (16-byte asynchronous copies, each thread waiting for its own), so that neither
// latency sits in the chain from one position to the next. 8 d bytes per position.
__global__ void __launch_bounds__(kVariantThreads) kernel_scan_kernel(const KernelScanParams p) {
  pdl_trigger();
  extern __shared__ __align__(16) float ks[];            // P [k][d] | v [k][d] | z ring | beta ring | lam_i | alpha_i[t]
  const int d = p.d, k = p.k;
  float* Ps = ks;
  float* vs = ks + (size_t)k * d;
  float* zr = vs + (size_t)k * d;
  float* br = zr + (size_t)kScanRing * d;
  float* l_s = br + (size_t)kScanRing * d;
  float* a_s = l_s + kKernelMixMaxK;
  if (threadIdx.x < k) l_s[threadIdx.x] = __ldg(p.lam + threadIdx.x);
  pdl_wait();
  const int64_t plane = p.Bp * (int64_t)d;
  for (int64_t b = blockIdx.x; b < p.Bp; b += gridDim.x) {
    __syncthreads();                                      // previous sample's slabs and rings are no longer read
    const float* zb = p.Z + b * p.n * (int64_t)d;
    float* yb = p.Y + b * p.n * (int64_t)d;
    const float* bb = p.beta + (int64_t)p.t0 * d;
    auto issue = [&](int jj) {                            // one group per position, empty past the end
      if (jj < p.n) {
        const int slot = jj % kScanRing;
        for (int e = threadIdx.x * 4; e < d; e += kVariantThreads * 4) {
          cp_async16(zr + (size_t)slot * d + e, zb + (int64_t)jj * d + e);
          cp_async16(br + (size_t)slot * d + e, bb + (int64_t)jj * d + e);
        }
      }
      cp_async_commit();
    };
#pragma unroll
    for (int jj = 0; jj < kScanRing - 1; ++jj) issue(jj);
    for (int e = threadIdx.x * 4; e < d; e += kVariantThreads * 4)
      for (int i = 0; i < k; ++i) st4(Ps + (size_t)i * d + e, ld4(p.P + (int64_t)i * plane + b * d + e));
    for (int j = 0; j < p.n; ++j) {
      issue(j + kScanRing - 1);                           // into the slot whose beta row was read one position ago
      cp_async_wait<kScanRing - 1>();                     // this thread's copies of position j have landed
      const int slot = j % kScanRing;
      if (threadIdx.x < k) a_s[threadIdx.x] = __ldg(p.alpha + (int64_t)threadIdx.x * p.n_ctx + p.t0 + j);
      for (int e = threadIdx.x * 4; e < d; e += kVariantThreads * 4) {
        const float4 z = ld4(zr + (size_t)slot * d + e);
        for (int i = 0; i < k; ++i) {
          float* Pi = Ps + (size_t)i * d + e;
          const float4 s = ld4(Pi);
          const float4 v = make_float4(z.x + s.x, z.y + s.y, z.z + s.z, z.w + s.w);
          st4(vs + (size_t)i * d + e, v);
          const float l = l_s[i];
          st4(Pi, make_float4(l * v.x, l * v.y, l * v.z, l * v.w));
        }
      }
      __syncthreads();                                    // v, alpha and everybody's beta copies of position j are visible
      const float* bt = br + (size_t)slot * d;
#pragma unroll 4
      for (int c = threadIdx.x; c < d; c += kVariantThreads) {
        float acc = bt[c];
        const int kk = d - c < k ? d - c : k;
        for (int i = 0; i < kk; ++i) acc = fmaf(a_s[i], vs[(size_t)i * d + c + i], acc);
        yb[(int64_t)j * d + c] = acc;
      }
      __syncthreads();
    }
    cp_async_wait<0>();
    for (int e = threadIdx.x * 4; e < d; e += kVariantThreads * 4)
      for (int i = 0; i < k; ++i) st4(p.P + (int64_t)i * plane + b * d + e, ld4(Ps + (size_t)i * d + e));
  }
}

}  // namespace srm
