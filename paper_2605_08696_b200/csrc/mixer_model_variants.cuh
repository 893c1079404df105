// Fused recurrent token-mixer step for models built from the two further mixers of the Architecture section:
// linearly combined heads (every head holds a row-repeat and a column-repeat matrix, Eq. 2 and Eq. 3 side by
// side, outputs combined with two weights per head; the cache is both sum terms, 2 d values per sample and
// layer) and non-unitary kernels (Eq. 11: k column-repeat filters, filter i applied to the hidden channels
// shifted by i, zero past the last channel; k d values per sample and layer).
//
// Same fusion as mixer_step_kernel: [x = E[tok]] -> LN1 -> cache update -> residual -> LN2 -> activation, one
// warp per row, the row in registers, 128-bit accesses. Lane l holds channels (32 i + l) 4 .. + 3 of vector i.
// The shifted reads of Eq. 11 never leave the warp: channel c + i of a filter's vector sits at most four lanes
// ahead (k <= 16), so every output float4 is put together from two shuffled float4s of the lanes ahead, the
// lanes at the end of a vector reading the start of the next one.
// Rows may be strided (x and a rows `x_stride` elements apart, tokens `tok_stride` apart): the sequence form of
// these models walks the positions of all prompts of a pass with this kernel, one launch per position, the
// cache staying in place between launches (it is the recurrence that defines the sequence form's result).
#pragma once

#include "common.cuh"
#include "mixer.cuh"

namespace srm {

struct VariantParams {
  float* x;              // row r at x + r * x_stride
  const int32_t* tok;    // token of row r at tok[r * tok_stride], or nullptr
  const void* E;
  void* S;               // cache planes [C][R_total, d] in the state type; plane c at S + c * plane (elements)
  void* a;               // row r at a + r * x_stride (activation type)
  const float* ln1_g; const float* ln1_b;
  const float* ln2_g; const float* ln2_b;
  const float* alpha;    // combined: row-repeat weights [h, n_ctx]; kernel: [k, n_ctx]
  const float* alpha_col;   // combined only: [h, n_ctx]
  const float* beta;     // [n_ctx, d]
  const float* lam;      // combined: row-repeat decays [h]; kernel: [k]
  const float* lam_col;  // combined only: [h]
  const float* w_comb;   // combined only: [h, 2]
  int64_t R, x_stride, tok_stride, plane;
  int d, h, k, n_ctx, t, vocab;
  float eps;
  uint32_t* status;
  const int32_t* ctr;    // device-side step counters or nullptr
};

// The float4 that lane (lane + delta) holds of vector j of the warp-distributed row f, the lanes past 31
// continuing in vector j + 1 and zeros following the last vector. 1 <= delta <= 4. Every lane calls it.
template <int NV>
__device__ __forceinline__ float4 fetch_ahead(const float4 (&f)[NV], int j, int delta, int lane) {
  const float4 nxt = (j + 1 < NV) ? f[(j + 1 < NV) ? j + 1 : j] : make_float4(0.f, 0.f, 0.f, 0.f);
  const float4 give = lane < delta ? nxt : f[j];       // lanes 0 .. delta-1 are read by the last lanes of the vector
  const int src = (lane + delta) & 31;
  return make_float4(__shfl_sync(0xffffffffu, give.x, src), __shfl_sync(0xffffffffu, give.y, src),
                     __shfl_sync(0xffffffffu, give.z, src), __shfl_sync(0xffffffffu, give.w, src));
}

// Channels c0 + i .. c0 + i + 3 of the row f, where c0 is the first channel this lane holds of vector j.
template <int NV>
__device__ __forceinline__ float4 shifted4(const float4 (&f)[NV], int j, int i, int lane) {
  const int q = i >> 2, s = i & 3;
  const float4 A = q == 0 ? f[j] : fetch_ahead<NV>(f, j, q, lane);
  if (s == 0) return A;                                // (i is the same in every lane: no divergence)
  const float4 B = fetch_ahead<NV>(f, j, q + 1, lane);
  if (s == 1) return make_float4(A.y, A.z, A.w, B.x);
  if (s == 2) return make_float4(A.z, A.w, B.x, B.y);
  return make_float4(A.w, B.x, B.y, B.z);
}

template <int NV, typename WT, typename ST, bool KERNEL_MIX>
__global__ void __launch_bounds__(kMixerWarps * 32) mixer_variant_step_kernel(const VariantParams p) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kMixerWarps + (threadIdx.x >> 5);
  if (row >= p.R) return;                              // (whole warps: the shuffles below stay converged)
  const int d = p.d;
  const int t = p.ctr != nullptr ? p.ctr[kCtrPos] : p.t;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);

  float4 v[NV];
  if (p.tok != nullptr) {
    int tk = p.tok[row * p.tok_stride];
    if (tk < 0 || tk >= p.vocab) {
      if (lane == 0) raise_status(p.status, kStatusTokenRange);
      tk = tk < 0 ? 0 : p.vocab - 1;
    }
    const WT* e = reinterpret_cast<const WT*>(p.E) + (int64_t)tk * d;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      v[i] = c < d ? ldg4(e + c) : zero;
    }
  } else {
    const float* xr = p.x + row * p.x_stride;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      v[i] = c < d ? ld4(xr + c) : zero;
    }
  }
  float mean, rstd;
  row_stats<NV>(v, lane, d, p.eps, mean, rstd);

  const float* beta_t = p.beta + (int64_t)t * d;
  ST* S0 = reinterpret_cast<ST*>(p.S) + row * d;
  float4 y[NV];
  if (!KERNEL_MIX) {
    // linearly combined heads:  y = w_row (alpha_row z + S_row) + w_col alpha_col (z + S_col) + beta_t
    //                           S_row <- lam_row (S_row + alpha_row z) ;  S_col <- lam_col (z + S_col)
    const int dh = d / p.h;
    ST* S1 = S0 + p.plane;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      y[i] = zero;
      if (c < d) {
        const float4 sr = ld4(S0 + c), sc = ld4(S1 + c);
        const float4 z = norm4(v[i], mean, rstd, ldg4(p.ln1_g + c), ldg4(p.ln1_b + c));
        const int g = c / dh;
        const float ar = __ldg(p.alpha + (int64_t)g * p.n_ctx + t), ac = __ldg(p.alpha_col + (int64_t)g * p.n_ctx + t);
        const float lr = __ldg(p.lam + g), lc = __ldg(p.lam_col + g);
        const float wr = __ldg(p.w_comb + 2 * g), wc = __ldg(p.w_comb + 2 * g + 1);
        const float4 bt = ldg4(beta_t + c);
        const float4 u = make_float4(ar * z.x, ar * z.y, ar * z.z, ar * z.w);
        const float4 w = make_float4(z.x + sc.x, z.y + sc.y, z.z + sc.z, z.w + sc.w);
        y[i] = make_float4(wr * (u.x + sr.x) + wc * (ac * w.x) + bt.x, wr * (u.y + sr.y) + wc * (ac * w.y) + bt.y,
                           wr * (u.z + sr.z) + wc * (ac * w.z) + bt.z, wr * (u.w + sr.w) + wc * (ac * w.w) + bt.w);
        st4(S0 + c, make_float4(lr * (sr.x + u.x), lr * (sr.y + u.y), lr * (sr.z + u.z), lr * (sr.w + u.w)));
        st4(S1 + c, make_float4(lc * w.x, lc * w.y, lc * w.z, lc * w.w));
      }
    }
  } else {
    // kernels of size k:  v_i = z + P_i ;  y[c] = beta_t[c] + sum_i alpha_i[t] v_i[c + i] (zero past channel d - 1) ;
    //                     P_i <- lam_i v_i
    // y starts as x + beta_t (the residual is folded in, so the row itself need not stay in registers); the cache
    // row of the NEXT filter is loaded before this filter's shuffles, so its latency overlaps them.
    float4 z[NV], f[NV], nx[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      z[i] = c < d ? norm4(v[i], mean, rstd, ldg4(p.ln1_g + c), ldg4(p.ln1_b + c)) : zero;
      if (c < d) {
        const float4 bt = ldg4(beta_t + c);
        y[i] = make_float4(v[i].x + bt.x, v[i].y + bt.y, v[i].z + bt.z, v[i].w + bt.w);
      } else {
        y[i] = zero;
      }
      f[i] = c < d ? ld4(S0 + c) : zero;                       // filter 0's cache row
    }
    for (int fi = 0; fi < p.k; ++fi) {
      const float al = __ldg(p.alpha + (int64_t)fi * p.n_ctx + t), lm = __ldg(p.lam + fi);
      ST* Pf = S0 + (int64_t)fi * p.plane;
      const bool more = fi + 1 < p.k;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int c = (i * 32 + lane) * 4;
        nx[i] = (more && c < d) ? ld4(Pf + p.plane + c) : zero;
      }
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int c = (i * 32 + lane) * 4;
        if (c < d) {
          const float4 w = make_float4(z[i].x + f[i].x, z[i].y + f[i].y, z[i].z + f[i].z, z[i].w + f[i].w);
          st4(Pf + c, make_float4(lm * w.x, lm * w.y, lm * w.z, lm * w.w));
          f[i] = make_float4(al * w.x, al * w.y, al * w.z, al * w.w);
        }
      }
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float4 sh = shifted4<NV>(f, i, fi, lane);
        y[i] = make_float4(y[i].x + sh.x, y[i].y + sh.y, y[i].z + sh.z, y[i].w + sh.w);
      }
#pragma unroll
      for (int i = 0; i < NV; ++i) f[i] = nx[i];
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = y[i];                  // x + y
  }

  float* xr = p.x + row * p.x_stride;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) {
      if (!KERNEL_MIX) v[i] = make_float4(v[i].x + y[i].x, v[i].y + y[i].y, v[i].z + y[i].z, v[i].w + y[i].w);
      st4(xr + c, v[i]);
    }
  }
  row_stats<NV>(v, lane, d, p.eps, mean, rstd);
  WT* ar = reinterpret_cast<WT*>(p.a) + row * p.x_stride;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) st4(ar + c, norm4(v[i], mean, rstd, ldg4(p.ln2_g + c), ldg4(p.ln2_b + c)));
  }
}

}  // namespace srm
