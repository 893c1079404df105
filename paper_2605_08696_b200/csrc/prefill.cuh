// Sequence-parallel token mixing over a prompt (Method/Architecture, Eq. 1 and Eq. 3).
//
// One CTA owns one sample and walks its n positions in tiles of T positions. Inside a tile the
// mixing is the explicit matrix product Y = Z M + B with the T x T diagonal block of M generated on
// the fly from alpha and lambda (row-repeat: M[i][j] = lambda^(j-i) alpha_i, column-repeat:
// lambda^(j-i) alpha_j, i <= j): each thread keeps its head's powers lambda^0..lambda^T in registers
// and the tile's alpha in shared memory, so the product needs no loads of M. The blocks of M above the diagonal are rank one, so their
// contribution is carried between tiles as the d-vector sum term of Eq. 2 / Eq. 3, which after
// the last tile is exactly the cache the recurrent form continues from. With T >= n this is the
// paper's full n x n product. LN1, the residual add and LN2 are fused around the mixing, so each
// row of the residual stream is read once and written once per layer.
#pragma once

#include "common.cuh"
#include "mixer.cuh"

namespace srm {

constexpr int kPrefillThreads = 256;
constexpr int kPrefillTile = 8;      // T: measured 16 -> 1304 us, 8 -> 784 us, 4 -> 1470 us for 512 prompts of 256 tokens at d = 1024
constexpr int kPrefillMaxHeads = 8;
constexpr int kPrefillMaxCPT = 8;    // channels per thread: d <= 2048

struct PrefillParams {
  float* x;              // [Bp*n, d] in/out
  const int32_t* tok;    // [Bp*n] or nullptr
  const void* E;
  void* S;               // [Bp, d] out (state type)
  void* a;               // [Bp*n, d] out (activation type)
  const float* ln1_g; const float* ln1_b;
  const float* ln2_g; const float* ln2_b;
  const float* alpha; const float* beta; const float* lam;
  int64_t Bp;
  int n, d, h, n_ctx, vocab;
  float eps;
  uint32_t* status;
  const int32_t* len;    // [Bp] prompt lengths (1 .. n; rows of a sample stay n apart), or nullptr: all prompts have n tokens
};

template <typename WT, typename ST>
__global__ void __launch_bounds__(kPrefillThreads) prefill_mixer_kernel(const PrefillParams p) {
  pdl_trigger();
  pdl_wait();
  constexpr int T = kPrefillTile;
  extern __shared__ float xs[];                       // [T][d] tile of the residual stream
  __shared__ float pw[kPrefillMaxHeads][T + 1];       // lambda^k
  __shared__ float al[kPrefillMaxHeads][T];           // alpha of the tile's positions
  __shared__ float mu[T], rs[T];                      // LN1 statistics of the tile's rows

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = p.d, stride = p.n, h = p.h, dh = d / h, h_row = h >> 1;
  const int64_t b = blockIdx.x;
  if (b >= p.Bp) return;
  int n = stride;                                      // positions of this sample
  if (p.len != nullptr) {
    n = p.len[b];
    if (n < 1 || n > stride) {
      if (tid == 0) raise_status(p.status, kStatusTokenRange);
      n = n < 1 ? 1 : stride;
    }
  }

  for (int i = tid; i < h * (T + 1); i += kPrefillThreads) {
    const int g = i / (T + 1), k = i % (T + 1);
    pw[g][k] = powf(__ldg(p.lam + g), (float)k);
  }
  float carry[kPrefillMaxCPT];
#pragma unroll
  for (int q = 0; q < kPrefillMaxCPT; ++q) carry[q] = 0.f;

  for (int j0 = 0; j0 < n; j0 += T) {
    const int rows = min(T, n - j0);
    const int64_t row0 = b * stride + j0;
    __syncthreads();     // previous tile fully written back before xs / Mt are overwritten
    // ---- load the tile (embedding rows for the first layer) ----
    if (p.tok != nullptr) {
      for (int r = warp; r < rows; r += kPrefillThreads / 32) {
        int tk = p.tok[row0 + r];
        if (tk < 0 || tk >= p.vocab) {
          if (lane == 0) raise_status(p.status, kStatusTokenRange);
          tk = tk < 0 ? 0 : p.vocab - 1;
        }
        const WT* e = reinterpret_cast<const WT*>(p.E) + (int64_t)tk * d;
        for (int c = lane * 4; c < d; c += 128) st4(xs + r * d + c, ldg4(e + c));
      }
    } else {
      const float* src = p.x + row0 * d;
      for (int i = tid * 4; i < rows * d; i += kPrefillThreads * 4) st4(xs + i, ld4(src + i));
    }
    for (int i = tid; i < h * T; i += kPrefillThreads) {
      const int g = i / T, r = i % T;
      al[g][r] = (r < rows) ? __ldg(p.alpha + (int64_t)g * p.n_ctx + j0 + r) : 0.f;
    }
    __syncthreads();
    // ---- LN1 statistics (one warp per row) ----
    for (int r = warp; r < rows; r += kPrefillThreads / 32) {
      const float* xr = xs + r * d;
      float s = 0.f;
      for (int c = lane * 4; c < d; c += 128) { const float4 v = ld4(xr + c); s += (v.x + v.y) + (v.z + v.w); }
      const float mean = warp_sum(s) / (float)d;
      float q = 0.f;
      for (int c = lane * 4; c < d; c += 128) {
        const float4 v = ld4(xr + c);
        const float t0 = v.x - mean, t1 = v.y - mean, t2 = v.z - mean, t3 = v.w - mean;
        q += (t0 * t0 + t1 * t1) + (t2 * t2 + t3 * t3);
      }
      const float rstd = rsqrtf(warp_sum(q) / (float)d + p.eps);
      if (lane == 0) { mu[r] = mean; rs[r] = rstd; }
    }
    __syncthreads();
    // ---- mixing: one thread per channel; z_i recomputed from x, mean, rstd ----
#pragma unroll
    for (int q = 0; q < kPrefillMaxCPT; ++q) {
      const int c = tid + q * kPrefillThreads;
      if (c < d) {
        const int g = c / dh;
        const bool is_row = g < h_row;
        const float gg = __ldg(p.ln1_g + c), bb = __ldg(p.ln1_b + c);
        // powers of this head's lambda and the tile's inputs u_i = alpha_i z_i (row-repeat) or z_i (column-repeat)
        float lp[T + 1];
#pragma unroll
        for (int k = 0; k <= T; ++k) lp[k] = pw[g][k];
        float u[T];
#pragma unroll
        for (int i = 0; i < T; ++i) {
          const float z = (i < rows) ? (xs[i * d + c] - mu[i]) * rs[i] * gg + bb : 0.f;
          u[i] = is_row ? al[g][i] * z : z;
        }
        const float S0 = carry[q];
#pragma unroll
        for (int j = 0; j < T; ++j) {
          if (j < rows) {
            // column j of the diagonal block: sum_i z_i M[i][j] with M[i][j] = lambda^(j-i) alpha_i (row)
            // or lambda^(j-i) alpha_j (column), plus the rank-one blocks above it folded into the carried sum
            float acc = lp[j] * S0;
#pragma unroll
            for (int i = 0; i <= j; ++i) acc = fmaf(u[i], lp[j - i], acc);
            if (!is_row) acc *= al[g][j];
            acc += __ldg(p.beta + (int64_t)(j0 + j) * d + c);
            xs[j * d + c] += acc;
          }
        }
        // sum term for the position after this tile (u_i = 0 beyond the last row of a ragged tile)
        float sn;
        if (rows == T) {
          sn = lp[T] * S0;
#pragma unroll
          for (int i = 0; i < T; ++i) sn = fmaf(lp[T - i], u[i], sn);
        } else {
          sn = pw[g][rows] * S0;
#pragma unroll
          for (int i = 0; i < T; ++i) {
            if (i < rows) sn = fmaf(pw[g][rows - i], u[i], sn);
          }
        }
        carry[q] = sn;
      }
    }
    __syncthreads();
    // ---- LN2 and write-back (one warp per row) ----
    for (int r = warp; r < rows; r += kPrefillThreads / 32) {
      const float* xr = xs + r * d;
      float s = 0.f;
      for (int c = lane * 4; c < d; c += 128) { const float4 v = ld4(xr + c); s += (v.x + v.y) + (v.z + v.w); }
      const float mean = warp_sum(s) / (float)d;
      float q = 0.f;
      for (int c = lane * 4; c < d; c += 128) {
        const float4 v = ld4(xr + c);
        const float t0 = v.x - mean, t1 = v.y - mean, t2 = v.z - mean, t3 = v.w - mean;
        q += (t0 * t0 + t1 * t1) + (t2 * t2 + t3 * t3);
      }
      const float rstd = rsqrtf(warp_sum(q) / (float)d + p.eps);
      float* xo = p.x + (row0 + r) * d;
      WT* ao = reinterpret_cast<WT*>(p.a) + (row0 + r) * d;
      for (int c = lane * 4; c < d; c += 128) {
        const float4 v = ld4(xr + c);
        st4(xo + c, v);
        st4(ao + c, norm4(v, mean, rstd, ldg4(p.ln2_g + c), ldg4(p.ln2_b + c)));
      }
    }
  }
  // positions beyond the sample's length: defined values for the GEMMs that follow (their results are not used)
  for (int64_t i = (int64_t)tid * 4; i < (int64_t)(stride - n) * d; i += kPrefillThreads * 4) {
    st4(p.x + (b * stride + n) * d + i, make_float4(0.f, 0.f, 0.f, 0.f));
    st4(reinterpret_cast<WT*>(p.a) + (b * stride + n) * d + i, make_float4(0.f, 0.f, 0.f, 0.f));
  }
  ST* So = reinterpret_cast<ST*>(p.S) + b * d;
#pragma unroll
  for (int q = 0; q < kPrefillMaxCPT; ++q) {
    const int c = tid + q * kPrefillThreads;
    if (c < d) So[c] = from_float<ST>(carry[q]);
  }
}

}  // namespace srm
