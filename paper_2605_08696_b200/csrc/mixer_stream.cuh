// Fused recurrent token-mixer step (Method/Architecture, Eq. 2 and Eq. 3, mixed heads), streaming version.
//
// Same arithmetic as mixer_step_kernel, other data movement. The warp-per-row kernel keeps 16 warps per
// SM and each of them walks the chain "load row -> LN1 -> load parameters -> update -> LN2 -> load
// parameters -> store" with every global latency exposed once per row. Here one persistent CTA per SM
//   - copies the per-layer parameters of this position (LN1/LN2 gain and shift, beta_t, alpha_t and lambda
//     per head) into shared memory once, before it orders itself behind the previous kernel (they are
//     weights: nothing in the stream writes them);
//   - gives every warp two row slots in shared memory and fills them with bulk asynchronous copies
//     (cp.async.bulk, completion counted on an mbarrier): the residual-stream row (or the embedding row of
//     the token for the first layer) and the cache row. A warp always has its next row in flight while it
//     works on the current one, so with W warps 2W rows (up to 192 KB) are in flight per SM;
//   - reads a row from shared memory into registers once, and writes x, the cache and the bf16 activation
//     straight to global memory with 128-bit stores, 512 contiguous bytes per warp instruction.
// With one position per row (MixerParams::pos, samples of different lengths) beta_t and alpha_t cannot be
// staged per CTA: each lane fetches its pieces of the row's beta_t (an L2 hit: the table is a few MB) and the
// head scalars with read-only loads, issued before the row's bulk copy is waited for.
// Requires d % 128 == 0 and a head width that is a multiple of 128 (every 128-channel vector lies in one
// head); other shapes take mixer_step_kernel. Every wait is bounded (status bit, then a clean exit).
#pragma once

#include "common.cuh"
#include "gemm_tc.cuh"   // mbarrier helpers
#include "mixer.cuh"     // MixerParams, row_stats_full

namespace srm {

constexpr int kStreamMaxWarps = 16;
constexpr int kStreamSmemBudget = 227 * 1024;

// global -> shared bulk copy (both addresses 16-byte aligned, size a multiple of 16) whose bytes are
// counted on an mbarrier of this CTA
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(tc::smem_u32(dst)), "l"(src), "r"(bytes), "r"(tc::smem_u32(bar))
               : "memory");
}

// dynamic shared memory: parameters (5 d floats + 16 head scalars) | W x 2 slots | 2 W mbarriers
__host__ __device__ inline size_t mixer_stream_param_bytes(int d) { return ((size_t)5 * d + 16) * 4; }
__host__ __device__ inline size_t mixer_stream_slot_bytes(int d, int state_elem) { return (size_t)d * 4 + (size_t)d * state_elem; }
inline int mixer_stream_warps(int d, int state_elem) {
  const size_t per_warp = 2 * mixer_stream_slot_bytes(d, state_elem) + 16;
  const size_t avail = kStreamSmemBudget - mixer_stream_param_bytes(d) - 64;
  const size_t w = avail / per_warp;
  return (int)(w > (size_t)kStreamMaxWarps ? kStreamMaxWarps : w);
}
inline size_t mixer_stream_smem(int d, int state_elem, int warps) {
  return mixer_stream_param_bytes(d) + (size_t)warps * (2 * mixer_stream_slot_bytes(d, state_elem) + 16) + 64;
}

template <int NV, typename WT, typename ST>
__global__ void __launch_bounds__(kStreamMaxWarps * 32, 1) mixer_stream_kernel(const MixerParams p) {
  pdl_trigger();
  extern __shared__ __align__(128) uint8_t sm[];
  const int d = p.d;
  const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* prm = reinterpret_cast<float*>(sm);                       // ln1_g | ln1_b | beta_t | ln2_g | ln2_b | alpha_t[8] lambda[8]
  float* heads = prm + 5 * d;
  const size_t x_bytes = (size_t)d * 4, s_bytes = (size_t)d * sizeof(ST), slot_bytes = x_bytes + s_bytes;
  uint8_t* slots = sm + mixer_stream_param_bytes(d);
  uint64_t* bars = reinterpret_cast<uint64_t*>(slots + (size_t)W * 2 * slot_bytes);

  // ---- parameters of this layer and position: constant data, fetched ahead of the dependency wait
  //      (unless the position comes from the device-side counter, which the previous step advanced) ----
  auto stage_params = [&](int t) {
    const float* beta_t = p.beta + (int64_t)t * d;
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
      st4(prm + i, ldg4(p.ln1_g + i));
      st4(prm + d + i, ldg4(p.ln1_b + i));
      st4(prm + 2 * d + i, ldg4(beta_t + i));
      st4(prm + 3 * d + i, ldg4(p.ln2_g + i));
      st4(prm + 4 * d + i, ldg4(p.ln2_b + i));
    }
    if (threadIdx.x < p.h) {
      heads[threadIdx.x] = __ldg(p.alpha + (int64_t)threadIdx.x * p.n_ctx + t);
      heads[8 + threadIdx.x] = __ldg(p.lam + threadIdx.x);
    }
  };
  if (p.ctr == nullptr) stage_params(p.t);
  if (threadIdx.x < 2 * W) tc::mbar_init(&bars[threadIdx.x], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();
  pdl_wait();
  if (p.ctr != nullptr) {
    stage_params(p.ctr[kCtrPos]);
    __syncthreads();
  }

  // ---- row schedule: CTA c owns rows c, c + G, c + 2G, ...; its i-th row goes to warp i % W ----
  const int64_t G = gridDim.x;
  const int64_t first = (int64_t)blockIdx.x + (int64_t)warp * G, stride = (int64_t)W * G;
  auto issue = [&](int j) {                 // lane 0: start the copies of this warp's j-th row
    const int64_t r = first + (int64_t)j * stride;
    if (r >= p.R) return;
    uint8_t* slot = slots + ((size_t)warp * 2 + (j & 1)) * slot_bytes;
    uint64_t* bar = &bars[warp * 2 + (j & 1)];
    const void* xsrc;
    uint32_t xb;
    if (p.tok != nullptr) {
      int tk = p.tok[r];
      if (tk < 0 || tk >= p.vocab) {
        raise_status(p.status, kStatusTokenRange);
        tk = tk < 0 ? 0 : p.vocab - 1;
      }
      xsrc = reinterpret_cast<const WT*>(p.E) + (int64_t)tk * d;
      xb = (uint32_t)(d * sizeof(WT));
    } else {
      xsrc = p.x + r * d;
      xb = (uint32_t)x_bytes;
    }
    tc::mbar_expect_tx(bar, xb + (uint32_t)s_bytes);
    bulk_g2s(slot, xsrc, xb, bar);
    bulk_g2s(slot + x_bytes, reinterpret_cast<const ST*>(p.S) + r * d, (uint32_t)s_bytes, bar);
  };
  if (lane == 0) { issue(0); issue(1); }

  const int c0 = lane * 4;
  const bool per_row = p.pos != nullptr;
  const int h_row = p.h >> 1;
  const int vph = (d / p.h) >> 7;           // 128-channel vectors per head
  const float inv_d = 1.0f / (float)d;
  bool ok = true;
  for (int j = 0;; ++j) {
    const int64_t r = first + (int64_t)j * stride;
    if (r >= p.R) break;
    uint8_t* slot = slots + ((size_t)warp * 2 + (j & 1)) * slot_bytes;
    // per-row position: its beta row and the head scalars come straight from global memory
    const int t_r = per_row ? min(max(p.pos[r], 0), p.n_ctx - 1) : 0;
    const float* beta_r = p.beta + (int64_t)t_r * d + c0;
    const float* alpha_r = p.alpha + t_r;
    if (!tc::mbar_wait(&bars[warp * 2 + (j & 1)], (uint32_t)(j >> 1) & 1u, p.status)) { ok = false; break; }

    float4 v[NV];
    if (p.tok != nullptr) {
      const WT* xs = reinterpret_cast<const WT*>(slot) + c0;
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] = ld4(xs + i * 128);
    } else {
      const float* xs = reinterpret_cast<const float*>(slot) + c0;
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] = ld4(xs + i * 128);
    }
    if (p.part != nullptr) {              // x + bias + plane 0 + plane 1 + ... (MixerParams::part)
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float4 bb = ldg4(p.part_bias + c0 + i * 128);
        v[i] = make_float4(v[i].x + bb.x, v[i].y + bb.y, v[i].z + bb.z, v[i].w + bb.w);
      }
      for (int s = 0; s < p.n_part; ++s) {
        const float* pr = p.part + (int64_t)s * p.part_plane + r * d + c0;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
          const float4 q = ld4(pr + i * 128);
          v[i] = make_float4(v[i].x + q.x, v[i].y + q.y, v[i].z + q.z, v[i].w + q.w);
        }
      }
    }
    float mean, rstd;
    row_stats_full<NV>(v, inv_d, p.eps, mean, rstd);
    const float nmr = -mean * rstd;                      // (x - mean) * rstd = x * rstd + nmr

    const ST* Ss = reinterpret_cast<const ST*>(slot + x_bytes) + c0;
    ST* Sg = reinterpret_cast<ST*>(p.S) + r * d + c0;
    float* xg = p.x + r * d + c0;
    int g = 0, left = vph;
    float al = per_row ? __ldg(alpha_r) : heads[0], lm = heads[8];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const float4 gg = ld4(prm + c0 + i * 128), bb = ld4(prm + d + c0 + i * 128);
      const float4 bt = per_row ? ldg4(beta_r + i * 128) : ld4(prm + 2 * d + c0 + i * 128);
      const float4 s = ld4(Ss + i * 128);
      float4 z;
      z.x = fmaf(fmaf(v[i].x, rstd, nmr), gg.x, bb.x); z.y = fmaf(fmaf(v[i].y, rstd, nmr), gg.y, bb.y);
      z.z = fmaf(fmaf(v[i].z, rstd, nmr), gg.z, bb.z); z.w = fmaf(fmaf(v[i].w, rstd, nmr), gg.w, bb.w);
      float4 y, sn;
      if (g < h_row) {            // row-repeat head, Eq. 2: y = a z + b + S ; S' = l (S + a z)
        const float4 u = make_float4(al * z.x, al * z.y, al * z.z, al * z.w);
        y = make_float4(u.x + bt.x + s.x, u.y + bt.y + s.y, u.z + bt.z + s.z, u.w + bt.w + s.w);
        sn = make_float4(lm * (s.x + u.x), lm * (s.y + u.y), lm * (s.z + u.z), lm * (s.w + u.w));
      } else {                    // column-repeat head, Eq. 3: y = a (z + S) + b ; S' = l (z + S)
        const float4 w = make_float4(z.x + s.x, z.y + s.y, z.z + s.z, z.w + s.w);
        y = make_float4(al * w.x + bt.x, al * w.y + bt.y, al * w.z + bt.z, al * w.w + bt.w);
        sn = make_float4(lm * w.x, lm * w.y, lm * w.z, lm * w.w);
      }
      st4(Sg + i * 128, sn);
      v[i] = make_float4(v[i].x + y.x, v[i].y + y.y, v[i].z + y.z, v[i].w + y.w);
      st4(xg + i * 128, v[i]);
      if (--left == 0 && i + 1 < NV) {                   // next vector starts the next head
        ++g; left = vph;
        al = per_row ? __ldg(alpha_r + (int64_t)g * p.n_ctx) : heads[g]; lm = heads[8 + g];
      }
    }
    // the slot has been read: order these generic-proxy reads before the next bulk copy into it
    tc::fence_async_smem();
    __syncwarp();
    if (lane == 0) issue(j + 2);

    row_stats_full<NV>(v, inv_d, p.eps, mean, rstd);
    const float nmr2 = -mean * rstd;
    WT* ar = reinterpret_cast<WT*>(p.a) + r * d + c0;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const float4 gg = ld4(prm + 3 * d + c0 + i * 128), bb = ld4(prm + 4 * d + c0 + i * 128);
      float4 o;
      o.x = fmaf(fmaf(v[i].x, rstd, nmr2), gg.x, bb.x); o.y = fmaf(fmaf(v[i].y, rstd, nmr2), gg.y, bb.y);
      o.z = fmaf(fmaf(v[i].z, rstd, nmr2), gg.z, bb.z); o.w = fmaf(fmaf(v[i].w, rstd, nmr2), gg.w, bb.w);
      st4(ar + i * 128, o);
    }
  }
  if (!ok) {
    // a copy never completed: give whatever is still in flight time to land before shared memory goes away
    const long long t0 = clock64();
    while (clock64() - t0 < (1ll << 21)) { }
  }
}

}  // namespace srm
