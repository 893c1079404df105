// Fused recurrent token-mixer step (Method/Architecture, Eq. 2 and Eq. 3, mixed heads) and the
// row-norm kernel. One warp owns one sample row of d channels and keeps it in registers: the
// row's residual stream and cache are each read once and written once with 128-bit accesses,
// 32 lanes covering 512 contiguous bytes per access.
#pragma once

#include "common.cuh"

namespace srm {

struct MixerParams {
  float* x;              // [R, d] residual stream, in/out
  const int32_t* tok;    // [R] or nullptr; when set, x starts from E[tok]
  const void* E;         // [V, d] embedding in the weight type
  void* S;               // [R, d] cache of this layer in the state type, in/out
  void* a;               // [R, d] LN2(x) in the activation type, out
  const float* ln1_g; const float* ln1_b;
  const float* ln2_g; const float* ln2_b;
  const float* alpha;    // [h, n_ctx]
  const float* beta;     // [n_ctx, d]
  const float* lam;      // [h]
  int64_t R;
  int d, h, n_ctx, t, vocab;
  float eps;
  uint32_t* status;
  const int32_t* ctr;    // device-side step counters, or nullptr: then `t` above is the position
  const int32_t* pos;    // [R] per-row positions (samples of different lengths), or nullptr: one position for all rows
  // mixer_stream_kernel only: partial products of the previous layer's down projection that have not been added into
  // x yet (the projection ran with its K dimension cut into n_part ranges, see GemmArgs::k_slices). The row this
  // kernel works on is x[r] + part_bias + part[0][r] + ... + part[n_part - 1][r], added in this order.
  const float* part = nullptr;        // [n_part] planes of part_plane elements, row r of a plane at r * d
  int n_part = 0;
  int64_t part_plane = 0;
  const float* part_bias = nullptr;   // [d]
};

// What a consumer adds to a row of the residual stream whose last down projection left partial products (see
// MixerParams::part); nullptr: nothing.
struct PartialSum {
  const float* part = nullptr;
  int n_part = 0;
  int64_t plane = 0;
  const float* bias = nullptr;
};

constexpr int kMixerWarps = 4;

// LayerNorm statistics of a register-resident row: two passes (mean, then centred variance).
template <int NV>
__device__ __forceinline__ void row_stats(const float4 (&v)[NV], int lane, int d, float eps,
                                          float& mean, float& rstd) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    if ((i * 32 + lane) * 4 < d) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  }
  mean = warp_sum(s) / (float)d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    if ((i * 32 + lane) * 4 < d) {
      float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, e = v[i].w - mean;
      q += (a * a + b * b) + (c * c + e * e);
    }
  }
  rstd = rsqrtf(warp_sum(q) / (float)d + eps);
}

__device__ __forceinline__ float4 norm4(float4 v, float mean, float rstd, float4 g, float4 b) {
  return make_float4((v.x - mean) * rstd * g.x + b.x, (v.y - mean) * rstd * g.y + b.y,
                     (v.z - mean) * rstd * g.z + b.z, (v.w - mean) * rstd * g.w + b.w);
}

// LayerNorm statistics when every lane holds NV full vectors (d == NV * 128).
template <int NV>
__device__ __forceinline__ void row_stats_full(const float4 (&v)[NV], float inv_d, float eps, float& mean, float& rstd) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  mean = warp_sum(s) * inv_d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, e = v[i].w - mean;
    q = fmaf(a, a, q); q = fmaf(b, b, q); q = fmaf(c, c, q); q = fmaf(e, e, q);
  }
  rstd = rsqrtf(warp_sum(q) * inv_d + eps);
}

// NV = ceil(d / 128): float4 vectors per lane. WT: weight/activation type, ST: cache type.
// General-shape version (any d that is a multiple of 4, any head width); shapes made of whole
// 128-channel vectors per head take mixer_stream_kernel instead.
template <int NV, typename WT, typename ST>
__global__ void __launch_bounds__(kMixerWarps * 32) mixer_step_kernel(const MixerParams p) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kMixerWarps + (threadIdx.x >> 5);
  if (row >= p.R) return;
  const int d = p.d;
  const int dh = d / p.h;
  const int h_row = p.h >> 1;
  const int t = p.pos != nullptr ? min(max(p.pos[row], 0), p.n_ctx - 1) : (p.ctr != nullptr ? p.ctr[kCtrPos] : p.t);

  float4 v[NV];
  if (p.tok != nullptr) {
    int tk = p.tok[row];
    if (tk < 0 || tk >= p.vocab) {
      if (lane == 0) raise_status(p.status, kStatusTokenRange);
      tk = tk < 0 ? 0 : p.vocab - 1;
    }
    const WT* e = reinterpret_cast<const WT*>(p.E) + (int64_t)tk * d;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      if (c < d) v[i] = ldg4(e + c);
    }
  } else {
    const float* xr = p.x + row * d;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      if (c < d) v[i] = ld4(xr + c);
    }
  }
  // issue the cache loads early so they overlap the LN1 reductions
  float4 s[NV];
  ST* Sr = reinterpret_cast<ST*>(p.S) + row * d;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) s[i] = ld4(Sr + c);
  }

  float mean, rstd;
  row_stats<NV>(v, lane, d, p.eps, mean, rstd);

  const float* beta_t = p.beta + (int64_t)t * d;
  float* xr = p.x + row * d;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) {
      const float4 z = norm4(v[i], mean, rstd, ldg4(p.ln1_g + c), ldg4(p.ln1_b + c));
      const int g = c / dh;
      const float al = __ldg(p.alpha + (int64_t)g * p.n_ctx + t);
      const float lm = __ldg(p.lam + g);
      const float4 bt = ldg4(beta_t + c);
      float4 y, sn;
      if (g < h_row) {            // row-repeat head, Eq. 2: y = a z + b + S ; S' = l (S + a z)
        const float4 u = make_float4(al * z.x, al * z.y, al * z.z, al * z.w);
        y = make_float4(u.x + bt.x + s[i].x, u.y + bt.y + s[i].y, u.z + bt.z + s[i].z, u.w + bt.w + s[i].w);
        sn = make_float4(lm * (s[i].x + u.x), lm * (s[i].y + u.y), lm * (s[i].z + u.z), lm * (s[i].w + u.w));
      } else {                    // column-repeat head, Eq. 3: y = a (z + S) + b ; S' = l (z + S)
        const float4 w = make_float4(z.x + s[i].x, z.y + s[i].y, z.z + s[i].z, z.w + s[i].w);
        y = make_float4(al * w.x + bt.x, al * w.y + bt.y, al * w.z + bt.z, al * w.w + bt.w);
        sn = make_float4(lm * w.x, lm * w.y, lm * w.z, lm * w.w);
      }
      st4(Sr + c, sn);
      v[i] = make_float4(v[i].x + y.x, v[i].y + y.y, v[i].z + y.z, v[i].w + y.w);
      st4(xr + c, v[i]);
    }
  }

  row_stats<NV>(v, lane, d, p.eps, mean, rstd);
  WT* ar = reinterpret_cast<WT*>(p.a) + row * d;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) st4(ar + c, norm4(v[i], mean, rstd, ldg4(p.ln2_g + c), ldg4(p.ln2_b + c)));
  }
}

// out[r, :] = LN(x[r * src_stride + src_offset, :]) in the activation type; with row_len the offset of row r
// is row_len[r] - 1 (the last position of a sample of that length).
template <int NV, typename WT>
__global__ void __launch_bounds__(kMixerWarps * 32)
norm_rows_kernel(const float* __restrict__ x, int64_t R, int64_t src_stride, int64_t src_offset,
                 const float* __restrict__ g, const float* __restrict__ b, float eps, int d,
                 WT* __restrict__ out, const int32_t* __restrict__ row_len, const PartialSum ps) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kMixerWarps + (threadIdx.x >> 5);
  if (row >= R) return;
  if (row_len != nullptr) src_offset = min(max((int64_t)row_len[row], (int64_t)1), src_stride) - 1;
  const float* xr = x + (row * src_stride + src_offset) * d;
  float4 v[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) v[i] = ld4(xr + c);
  }
  if (ps.part != nullptr) {              // x + bias + plane 0 + plane 1 + ... (row r of every plane)
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = (i * 32 + lane) * 4;
      if (c < d) {
        const float4 bb = ldg4(ps.bias + c);
        v[i] = make_float4(v[i].x + bb.x, v[i].y + bb.y, v[i].z + bb.z, v[i].w + bb.w);
      }
    }
    for (int s = 0; s < ps.n_part; ++s) {
      const float* pr = ps.part + (int64_t)s * ps.plane + row * d;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int c = (i * 32 + lane) * 4;
        if (c < d) {
          const float4 q = ld4(pr + c);
          v[i] = make_float4(v[i].x + q.x, v[i].y + q.y, v[i].z + q.z, v[i].w + q.w);
        }
      }
    }
  }
  float mean, rstd;
  row_stats<NV>(v, lane, d, eps, mean, rstd);
  WT* o = out + row * d;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = (i * 32 + lane) * 4;
    if (c < d) st4(o + c, norm4(v[i], mean, rstd, ldg4(g + c), ldg4(b + c)));
  }
}

}  // namespace srm
