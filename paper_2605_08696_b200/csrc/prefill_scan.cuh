// Token mixing over whole prompts as a scan (Method/Architecture: the matrix M of Eq. 1 / Eq. 3 applied through
// its recurrence, Eq. 2 / Eq. 3 right-hand sides; the paper names a scan for the prefill as an open option).
//
// prefill_mixer_kernel multiplies by the diagonal blocks of M explicitly, one CTA per sample, five block
// barriers per tile of eight positions; with many prompts in flight that kernel, not the GEMMs around it, was
// 43 % of the prefill. Here one WARP owns a sample and walks its positions in order, exactly like the decode
// kernel walks rows, except that the cache never leaves the registers: per position it reads the row of the
// residual stream (staged in shared memory by a bulk copy issued two positions ahead), normalises (LN1),
// applies y_j = alpha_j z_j + beta_j + S, S <- lambda (S + alpha_j z_j) (row-repeat heads) or
// y_j = alpha_j (z_j + S) + beta_j, S <- lambda (z_j + S) (column-repeat heads), adds y to the row,
// normalises again (LN2) and writes the row and its bf16 activation. The d-vector S after the last position is
// the cache the recurrent form continues from. Bytes per position: d * (4 + 4 + 2); no barrier in the loop.
// The positions of one sample are sequential, so the kernel wants at least as many samples as the GPU has warp
// slots for it (about 2000); with few prompts prefill_mixer_kernel is the faster one, and the host chooses.
// Same shape requirements as mixer_stream_kernel (whole 128-channel vectors per head).
#pragma once

#include "common.cuh"
#include "gemm_tc.cuh"        // mbarrier helpers
#include "mixer.cuh"          // row_stats_full
#include "mixer_stream.cuh"   // bulk_g2s
#include "prefill.cuh"        // PrefillParams

namespace srm {

constexpr int kScanSmemBudget = 227 * 1024;
__host__ __device__ inline int prefill_scan_max_warps(int nv) { return nv <= 8 ? 16 : 8; }   // register budget: v and S per lane
inline int prefill_scan_warps(int d, int64_t samples, int num_sms) {
  const size_t per_warp = 2 * (size_t)d * 4 + 16, fixed = (size_t)4 * d * 4 + 64 + 64;
  int w = (int)((kScanSmemBudget - fixed) / per_warp);
  const int cap = prefill_scan_max_warps(d / 128);
  if (w > cap) w = cap;
  const int64_t need = (samples + num_sms - 1) / num_sms;          // samples per SM
  if (need < w) w = (int)(need < 1 ? 1 : need);
  return w;
}
inline size_t prefill_scan_smem(int d, int warps) { return (size_t)4 * d * 4 + 64 + (size_t)warps * (2 * (size_t)d * 4 + 16) + 64; }

template <int NV, typename WT, typename ST>
__global__ void __launch_bounds__(NV <= 8 ? 512 : 256, 1) prefill_scan_kernel(const PrefillParams p) {
  pdl_trigger();
  extern __shared__ __align__(128) uint8_t sm[];
  const int d = p.d;
  const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* prm = reinterpret_cast<float*>(sm);                        // ln1_g | ln1_b | ln2_g | ln2_b | lambda[8]
  float* lam_s = prm + 4 * d;
  const size_t x_bytes = (size_t)d * 4;
  uint8_t* slots = sm + (size_t)4 * d * 4 + 64;
  uint64_t* bars = reinterpret_cast<uint64_t*>(slots + (size_t)W * 2 * x_bytes);

  // layer parameters: constant data, fetched ahead of the dependency wait
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    st4(prm + i, ldg4(p.ln1_g + i));
    st4(prm + d + i, ldg4(p.ln1_b + i));
    st4(prm + 2 * d + i, ldg4(p.ln2_g + i));
    st4(prm + 3 * d + i, ldg4(p.ln2_b + i));
  }
  if (threadIdx.x < p.h) lam_s[threadIdx.x] = __ldg(p.lam + threadIdx.x);
  if (threadIdx.x < 2 * W) tc::mbar_init(&bars[threadIdx.x], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();
  pdl_wait();

  const int c0 = lane * 4;
  const int h_row = p.h >> 1;
  const int vph = (d / p.h) >> 7;
  const float inv_d = 1.0f / (float)d;
  const int stride = p.n;
  uint32_t k = 0;                             // rows this warp has consumed: slot k & 1, barrier parity (k >> 1) & 1
  bool ok = true;
  for (int64_t b = (int64_t)blockIdx.x + (int64_t)warp * gridDim.x; ok && b < p.Bp; b += (int64_t)W * gridDim.x) {
    int n = stride;
    if (p.len != nullptr) {
      n = p.len[b];
      if (n < 1 || n > stride) {
        if (lane == 0) raise_status(p.status, kStatusTokenRange);
        n = n < 1 ? 1 : stride;
      }
    }
    const int64_t row0 = b * stride;
    auto issue = [&](int j, uint32_t kk) {     // lane 0: start the copy of position j into the slot of row count kk
      if (j >= n) return;
      uint8_t* slot = slots + ((size_t)warp * 2 + (kk & 1)) * x_bytes;
      uint64_t* bar = &bars[warp * 2 + (kk & 1)];
      const void* src;
      uint32_t nb;
      if (p.tok != nullptr) {
        int tk = p.tok[row0 + j];
        if (tk < 0 || tk >= p.vocab) {
          raise_status(p.status, kStatusTokenRange);
          tk = tk < 0 ? 0 : p.vocab - 1;
        }
        src = reinterpret_cast<const WT*>(p.E) + (int64_t)tk * d;
        nb = (uint32_t)(d * sizeof(WT));
      } else {
        src = p.x + (row0 + j) * d;
        nb = (uint32_t)x_bytes;
      }
      tc::mbar_expect_tx(bar, nb);
      bulk_g2s(slot, src, nb, bar);
    };
    if (lane == 0) { issue(0, k); issue(1, k + 1); }

    float4 S[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) S[i] = make_float4(0.f, 0.f, 0.f, 0.f);

    for (int j = 0; j < n; ++j, ++k) {
      uint8_t* slot = slots + ((size_t)warp * 2 + (k & 1)) * x_bytes;
      const float* beta_j = p.beta + (int64_t)j * d + c0;
      const float* alpha_j = p.alpha + j;
      if (!tc::mbar_wait(&bars[warp * 2 + (k & 1)], (k >> 1) & 1u, p.status)) { ok = false; break; }

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
      // the slot has been read: order these generic-proxy reads before the next bulk copy into it
      tc::fence_async_smem();
      __syncwarp();
      if (lane == 0) issue(j + 2, k + 2);

      float mean, rstd;
      row_stats_full<NV>(v, inv_d, p.eps, mean, rstd);
      const float nmr = -mean * rstd;
      float* xg = p.x + (row0 + j) * d + c0;
      int g = 0, left = vph;
      float al = __ldg(alpha_j), lm = lam_s[0];
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float4 gg = ld4(prm + c0 + i * 128), bb = ld4(prm + d + c0 + i * 128);
        const float4 bt = ldg4(beta_j + i * 128);
        const float4 s = S[i];
        float4 z;
        z.x = fmaf(fmaf(v[i].x, rstd, nmr), gg.x, bb.x); z.y = fmaf(fmaf(v[i].y, rstd, nmr), gg.y, bb.y);
        z.z = fmaf(fmaf(v[i].z, rstd, nmr), gg.z, bb.z); z.w = fmaf(fmaf(v[i].w, rstd, nmr), gg.w, bb.w);
        float4 y;
        if (g < h_row) {            // row-repeat head, Eq. 2
          const float4 u = make_float4(al * z.x, al * z.y, al * z.z, al * z.w);
          y = make_float4(u.x + bt.x + s.x, u.y + bt.y + s.y, u.z + bt.z + s.z, u.w + bt.w + s.w);
          S[i] = make_float4(lm * (s.x + u.x), lm * (s.y + u.y), lm * (s.z + u.z), lm * (s.w + u.w));
        } else {                    // column-repeat head, Eq. 3
          const float4 w = make_float4(z.x + s.x, z.y + s.y, z.z + s.z, z.w + s.w);
          y = make_float4(al * w.x + bt.x, al * w.y + bt.y, al * w.z + bt.z, al * w.w + bt.w);
          S[i] = make_float4(lm * w.x, lm * w.y, lm * w.z, lm * w.w);
        }
        v[i] = make_float4(v[i].x + y.x, v[i].y + y.y, v[i].z + y.z, v[i].w + y.w);
        st4(xg + i * 128, v[i]);
        if (--left == 0 && i + 1 < NV) {
          ++g; left = vph;
          al = __ldg(alpha_j + (int64_t)g * p.n_ctx); lm = lam_s[g];
        }
      }
      row_stats_full<NV>(v, inv_d, p.eps, mean, rstd);
      const float nmr2 = -mean * rstd;
      WT* ar = reinterpret_cast<WT*>(p.a) + (row0 + j) * d + c0;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float4 gg = ld4(prm + 2 * d + c0 + i * 128), bb = ld4(prm + 3 * d + c0 + i * 128);
        float4 o;
        o.x = fmaf(fmaf(v[i].x, rstd, nmr2), gg.x, bb.x); o.y = fmaf(fmaf(v[i].y, rstd, nmr2), gg.y, bb.y);
        o.z = fmaf(fmaf(v[i].z, rstd, nmr2), gg.z, bb.z); o.w = fmaf(fmaf(v[i].w, rstd, nmr2), gg.w, bb.w);
        st4(ar + i * 128, o);
      }
    }
    if (!ok) break;
    // the cache the recurrent form continues from
    ST* So = reinterpret_cast<ST*>(p.S) + b * d + c0;
#pragma unroll
    for (int i = 0; i < NV; ++i) st4(So + i * 128, S[i]);
    // positions beyond the sample's length: defined values for the GEMMs that follow (their results are not used)
    for (int j = n; j < stride; ++j) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        st4(p.x + (row0 + j) * d + c0 + i * 128, make_float4(0.f, 0.f, 0.f, 0.f));
        st4(reinterpret_cast<WT*>(p.a) + (row0 + j) * d + c0 + i * 128, make_float4(0.f, 0.f, 0.f, 0.f));
      }
    }
  }
  if (!ok) {
    const long long t0 = clock64();
    while (clock64() - t0 < (1ll << 21)) { }
  }
}

}  // namespace srm
