// Token mixer with head projections (Method/Architecture, Eq. 10):
//   Y = P_out (concat_g [(I_g X) M_g + beta_g]).
// The two projections are GEMMs (W_in stacks the I_g, W_out = P_out) run by the tensor-core kernel; what is
// left between them works on the PROJECTED values q = W_in LN1(x), has no reduction over channels, and is
// written here: the recurrent update of one position (decode) and the sequence-parallel product (prefill).
// Both are pure streams: every thread owns four adjacent channels, which never straddle a head.
#pragma once

#include "common.cuh"

namespace srm {

struct MixProjParams {
  const float* q;        // [rows, d] projected inputs (fp32, output of the W_in GEMM)
  void* S;               // decode: [R, d] cache in/out; prefill: [Bp, d] cache out (state type)
  void* y;               // [rows, d] mixed heads, concatenated, in the activation type (input of the W_out GEMM)
  const float* alpha;    // [h, n_ctx]
  const float* beta;     // [n_ctx, d]
  const float* lam;      // [h]
  int64_t R;             // decode: rows; prefill: samples
  int d, h, n_ctx;
  int t;                 // decode: position
  int n;                 // prefill: prompt length
  const int32_t* ctr;    // decode: device-side step counters, or nullptr: then `t` is the position
  const int32_t* pos;    // decode: [R] per-row positions, or nullptr; prefill: [R] prompt lengths (<= n), or nullptr
  uint32_t* status;      // device status word (a prompt length outside [1, n] is clamped and flagged)
};

constexpr int kMixProjThreads = 256;

// x[r, :] = E[tok[r], :] in fp32 (first layer of the projected path; token ids are clamped and flagged).
template <typename WT>
__global__ void __launch_bounds__(kMixProjThreads)
embed_rows_kernel(const int32_t* __restrict__ tok, const WT* __restrict__ E, float* __restrict__ x, int64_t R, int d,
                  int vocab, uint32_t* status) {
  pdl_trigger();
  pdl_wait();
  const int64_t vec = (int64_t)blockIdx.x * kMixProjThreads + threadIdx.x;     // one float4 per thread
  const int vpr = d >> 2;
  if (vec >= R * vpr) return;
  const int64_t r = vec / vpr;
  const int c = (int)(vec % vpr) * 4;
  int tk = tok[r];
  if (tk < 0 || tk >= vocab) {
    if (c == 0) raise_status(status, kStatusTokenRange);
    tk = tk < 0 ? 0 : vocab - 1;
  }
  st4(x + r * d + c, ldg4(E + (int64_t)tk * d + c));
}

// Decode, position t (Eq. 2 / Eq. 3 on projected values): row head  y = a q + S + b ; S' = l (S + a q),
// column head  y = a (q + S) + b ; S' = l (q + S).
template <typename WT, typename ST>
__global__ void __launch_bounds__(kMixProjThreads) mixer_proj_step_kernel(const MixProjParams p) {
  pdl_trigger();
  pdl_wait();
  const int64_t vec = (int64_t)blockIdx.x * kMixProjThreads + threadIdx.x;
  const int vpr = p.d >> 2;
  if (vec >= p.R * vpr) return;
  const int64_t r = vec / vpr;
  const int c = (int)(vec % vpr) * 4;
  const int g = c / (p.d / p.h);
  const int t = p.pos != nullptr ? min(max(p.pos[r], 0), p.n_ctx - 1) : (p.ctr != nullptr ? p.ctr[kCtrPos] : p.t);
  const float al = __ldg(p.alpha + (int64_t)g * p.n_ctx + t), lm = __ldg(p.lam + g);
  const float4 bt = ldg4(p.beta + (int64_t)t * p.d + c);
  const float4 q = ld4(p.q + r * p.d + c);
  ST* Sp = reinterpret_cast<ST*>(p.S) + r * p.d + c;
  const float4 s = ld4(Sp);
  float4 y, sn;
  if (g < (p.h >> 1)) {
    const float4 u = make_float4(al * q.x, al * q.y, al * q.z, al * q.w);
    y = make_float4(u.x + bt.x + s.x, u.y + bt.y + s.y, u.z + bt.z + s.z, u.w + bt.w + s.w);
    sn = make_float4(lm * (s.x + u.x), lm * (s.y + u.y), lm * (s.z + u.z), lm * (s.w + u.w));
  } else {
    const float4 w = make_float4(q.x + s.x, q.y + s.y, q.z + s.z, q.w + s.w);
    y = make_float4(al * w.x + bt.x, al * w.y + bt.y, al * w.z + bt.z, al * w.w + bt.w);
    sn = make_float4(lm * w.x, lm * w.y, lm * w.z, lm * w.w);
  }
  st4(Sp, sn);
  st4(reinterpret_cast<WT*>(p.y) + r * p.d + c, y);
}

// Prefill: the sequence-parallel product along the n positions of one sample (Eq. 1 / Eq. 3 on projected
// values), four channels per thread. Positions are taken in tiles of T: inside a tile the T x T diagonal
// block of M (entries lambda^(j-i) alpha_i, or alpha_j, generated from register-resident powers of lambda)
// multiplies the tile's inputs explicitly; the blocks above the diagonal are rank one and enter through the
// carried sum term, which after the last tile is the cache. Rows of q and y are read and written once.
constexpr int kMixProjTile = 8;

template <typename WT, typename ST>
__global__ void __launch_bounds__(kMixProjThreads) mixer_proj_prefill_kernel(const MixProjParams p) {
  constexpr int T = kMixProjTile;
  pdl_trigger();
  pdl_wait();
  const int64_t vec = (int64_t)blockIdx.x * kMixProjThreads + threadIdx.x;
  const int vpr = p.d >> 2;
  if (vec >= p.R * vpr) return;
  const int64_t b = vec / vpr;
  const int c = (int)(vec % vpr) * 4;
  const int g = c / (p.d / p.h);
  const bool is_row = g < (p.h >> 1);
  const float lm = __ldg(p.lam + g);
  float lp[T];                       // lambda^0 .. lambda^(T-1)
  lp[0] = 1.f;
#pragma unroll
  for (int k = 1; k < T; ++k) lp[k] = lp[k - 1] * lm;
  const float* al = p.alpha + (int64_t)g * p.n_ctx;
  float4 carry = make_float4(0.f, 0.f, 0.f, 0.f);
  const int nb = p.pos != nullptr ? min(max(p.pos[b], 1), p.n) : p.n;      // this sample's length; rows stay n apart
  if (p.pos != nullptr && c == 0 && p.pos[b] != nb) raise_status(p.status, kStatusTokenRange);
  for (int j0 = 0; j0 < nb; j0 += T) {
    const int rows = min(T, nb - j0);
    float4 u[T];
    float a[T];
#pragma unroll
    for (int i = 0; i < T; ++i) {
      a[i] = (i < rows) ? __ldg(al + j0 + i) : 0.f;
      u[i] = (i < rows) ? ld4(p.q + (b * p.n + j0 + i) * p.d + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      if (is_row) u[i] = make_float4(a[i] * u[i].x, a[i] * u[i].y, a[i] * u[i].z, a[i] * u[i].w);
    }
#pragma unroll
    for (int j = 0; j < T; ++j) {
      if (j < rows) {
        // carry is the sum term the tile's first position reads; position j reads lambda^j of it
        float4 acc = make_float4(lp[j] * carry.x, lp[j] * carry.y, lp[j] * carry.z, lp[j] * carry.w);
#pragma unroll
        for (int i = 0; i <= j; ++i) {
          acc.x = fmaf(u[i].x, lp[j - i], acc.x); acc.y = fmaf(u[i].y, lp[j - i], acc.y);
          acc.z = fmaf(u[i].z, lp[j - i], acc.z); acc.w = fmaf(u[i].w, lp[j - i], acc.w);
        }
        if (!is_row) acc = make_float4(a[j] * acc.x, a[j] * acc.y, a[j] * acc.z, a[j] * acc.w);
        const float4 bt = ldg4(p.beta + (int64_t)(j0 + j) * p.d + c);
        acc = make_float4(acc.x + bt.x, acc.y + bt.y, acc.z + bt.z, acc.w + bt.w);
        st4(reinterpret_cast<WT*>(p.y) + (b * p.n + j0 + j) * p.d + c, acc);
      }
    }
    // carried term after this tile: carry' = sum_{i < rows} lambda^(rows - i) u_i + lambda^rows carry,
    // built position by position so that a ragged last tile needs no dynamic register indexing
#pragma unroll
    for (int i = 0; i < T; ++i) {
      if (i < rows) {
        carry = make_float4(lm * (carry.x + u[i].x), lm * (carry.y + u[i].y), lm * (carry.z + u[i].z),
                            lm * (carry.w + u[i].w));
      }
    }
  }
  for (int j = nb; j < p.n; ++j)          // positions beyond the sample's length: defined values for the GEMM that follows
    st4(reinterpret_cast<WT*>(p.y) + (b * p.n + j) * p.d + c, make_float4(0.f, 0.f, 0.f, 0.f));
  st4(reinterpret_cast<ST*>(p.S) + b * p.d + c, carry);
}

}  // namespace srm
