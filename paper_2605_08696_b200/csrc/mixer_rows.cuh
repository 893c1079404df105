// Fused recurrent token-mixer step (Method/Architecture, Eq. 2 and Eq. 3, mixed heads): one CTA per row.
//
// Same arithmetic as mixer_step_kernel / mixer_stream_kernel, other distribution of the work. Those kernels give a
// row to one warp, which then owns 8 to 16 vectors per lane and must fetch the five per-channel parameter vectors
// again for every row; with the row staged in shared memory only 8 to 12 warps fit on an SM, and the kernel ends up
// bound by the latency of its own instruction stream (IPC 1.2). Here thread i of a CTA owns channels 4 i .. 4 i + 3
// of EVERY row the CTA walks, so LN1 / LN2 gain and shift, the decay and (with one position for all rows) beta_t
// and alpha_t sit in registers for the whole kernel; a row costs two 16-byte loads and three 16-byte stores per
// thread, the LayerNorm statistics are sums over the CTA (warp shuffles, one shared-memory word per warp, one
// barrier per sum), and the next row's loads are in flight while the current one is reduced. The CTAs are small
// (d / 4 threads, a few dozen registers, 256 bytes of shared memory), so eight of them share an SM and hide each
// other's barriers. Any d that is a multiple of 4 with heads that are a multiple of 4 wide; d <= 4096.
#pragma once

#include "common.cuh"
#include "mixer.cuh"

namespace srm {

constexpr int kRowsMaxWarps = 32;

// Sum of one value per thread over the CTA; every thread calls it. `red` is [2][kRowsMaxWarps]: consecutive sums
// alternate between the halves, so one barrier per sum suffices (a half is rewritten two sums later, and every
// thread has passed the barrier in between only after reading it).
__device__ __forceinline__ float cta_sum_alt(float v, float (*red)[kRowsMaxWarps], int& phase, int nw) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) red[phase][threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < nw; ++w) t += red[phase][w];
  phase ^= 1;
  return t;
}

template <typename WT, typename ST>
__global__ void __launch_bounds__(1024) mixer_rows_kernel(const MixerParams p) {
  pdl_trigger();
  __shared__ float red[2][kRowsMaxWarps];
  const int d = p.d, c = threadIdx.x * 4, nw = blockDim.x >> 5;
  const bool on = c < d;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  const int g = on ? c / (d / p.h) : 0;
  const bool row_head = g < (p.h >> 1);
  const bool per_row = p.pos != nullptr;
  // ---- parameters of this thread's channels: weights, fetched ahead of the dependency wait ----
  float4 g1 = zero, b1 = zero, g2 = zero, b2 = zero, bt = zero;
  float al = 0.f, lm = 0.f;
  if (on) {
    g1 = ldg4(p.ln1_g + c); b1 = ldg4(p.ln1_b + c); g2 = ldg4(p.ln2_g + c); b2 = ldg4(p.ln2_b + c);
    lm = __ldg(p.lam + g);
    if (!per_row && p.ctr == nullptr) {
      bt = ldg4(p.beta + (int64_t)p.t * d + c);
      al = __ldg(p.alpha + (int64_t)g * p.n_ctx + p.t);
    }
  }
  pdl_wait();
  if (on && !per_row && p.ctr != nullptr) {            // the position comes from the device-side counter
    const int t = p.ctr[kCtrPos];
    bt = ldg4(p.beta + (int64_t)t * d + c);
    al = __ldg(p.alpha + (int64_t)g * p.n_ctx + t);
  }
  const float inv_d = 1.0f / (float)d;
  int phase = 0;

  // x (or the embedding row of the token) and the cache row of row r, for this thread's channels
  auto load_row = [&](int64_t r, float4& v, float4& s) {
    if (!on) return;
    if (p.tok != nullptr) {
      int tk = p.tok[r];
      if (tk < 0 || tk >= p.vocab) {
        if (threadIdx.x == 0) raise_status(p.status, kStatusTokenRange);
        tk = tk < 0 ? 0 : p.vocab - 1;
      }
      v = ldg4(reinterpret_cast<const WT*>(p.E) + (int64_t)tk * d + c);
    } else {
      v = ld4(p.x + r * d + c);
    }
    s = ld4(reinterpret_cast<const ST*>(p.S) + r * d + c);
  };

  float4 v = zero, s = zero;
  int64_t r = blockIdx.x;
  if (r < p.R) load_row(r, v, s);
  for (; r < p.R; r += gridDim.x) {
    const int64_t rn = r + gridDim.x;
    float4 vn = zero, sn_ = zero;
    if (rn < p.R) load_row(rn, vn, sn_);               // the next row is on its way while this one is reduced
    if (per_row && on) {
      const int t = min(max(p.pos[r], 0), p.n_ctx - 1);
      bt = ldg4(p.beta + (int64_t)t * d + c);
      al = __ldg(p.alpha + (int64_t)g * p.n_ctx + t);
    }
    float mean = cta_sum_alt((v.x + v.y) + (v.z + v.w), red, phase, nw) * inv_d;
    float4 cd = on ? make_float4(v.x - mean, v.y - mean, v.z - mean, v.w - mean) : zero;
    float rstd = rsqrtf(cta_sum_alt((cd.x * cd.x + cd.y * cd.y) + (cd.z * cd.z + cd.w * cd.w), red, phase, nw) * inv_d + p.eps);
    if (on) {
      const float4 z = norm4(v, mean, rstd, g1, b1);
      float4 y, sn;
      if (row_head) {             // row-repeat head, Eq. 2: y = a z + b + S ; S' = l (S + a z)
        const float4 u = make_float4(al * z.x, al * z.y, al * z.z, al * z.w);
        y = make_float4(u.x + bt.x + s.x, u.y + bt.y + s.y, u.z + bt.z + s.z, u.w + bt.w + s.w);
        sn = make_float4(lm * (s.x + u.x), lm * (s.y + u.y), lm * (s.z + u.z), lm * (s.w + u.w));
      } else {                    // column-repeat head, Eq. 3: y = a (z + S) + b ; S' = l (z + S)
        const float4 q = make_float4(z.x + s.x, z.y + s.y, z.z + s.z, z.w + s.w);
        y = make_float4(al * q.x + bt.x, al * q.y + bt.y, al * q.z + bt.z, al * q.w + bt.w);
        sn = make_float4(lm * q.x, lm * q.y, lm * q.z, lm * q.w);
      }
      st4(reinterpret_cast<ST*>(p.S) + r * d + c, sn);
      v = make_float4(v.x + y.x, v.y + y.y, v.z + y.z, v.w + y.w);
      st4(p.x + r * d + c, v);
    }
    mean = cta_sum_alt((v.x + v.y) + (v.z + v.w), red, phase, nw) * inv_d;
    cd = on ? make_float4(v.x - mean, v.y - mean, v.z - mean, v.w - mean) : zero;
    rstd = rsqrtf(cta_sum_alt((cd.x * cd.x + cd.y * cd.y) + (cd.z * cd.z + cd.w * cd.w), red, phase, nw) * inv_d + p.eps);
    if (on) st4(reinterpret_cast<WT*>(p.a) + r * d + c, norm4(v, mean, rstd, g2, b2));
    v = vn; s = sn_;
  }
}

}  // namespace srm
