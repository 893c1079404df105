// One decode step of a SMALL batch (at most 64 samples) as a single persistent kernel.
//
// With a handful of rows the step is bound by reading the weights once (the mid model: 467 MB, 70 us at HBM
// speed) and by the latency of its 50 dependent kernels, not by arithmetic: a 256 x 256 tensor-core tile keeps 4
// to 16 of the 74 CTA pairs busy on a one-row GEMM, and every launch costs its ramp. Here the whole step --
// embedding, L x (token-mixer cache update [Eq. 2, Eq. 3], feed-forward up and down), final norm, LM head,
// greedy selection -- runs in ONE cooperative kernel of one CTA per SM. Every dense projection is cut into
// column slabs (and, for the down projection, k-slabs), one per CTA, so that all SMs stream weights at once;
// the few activation rows are re-read by every CTA from L2. Phases are separated by grid-wide barriers; a CTA
// starts the bulk copy of its NEXT weight slab before it waits at a barrier (weights are constant), so the
// weight stream continues across the barriers. The contractions run on mma.sync (m16n8k16, bf16 in, fp32
// accumulate): with M <= 64 the kernel is HBM-bound and a tcgen05 tile would be mostly padding.
//
// The down projection's k-slabs leave partial sums in scratch memory; the next phase (the following layer's
// mixer, or the final norm) adds them in slab order, so results do not depend on timing.
// Every wait (grid barrier, mbarrier) is bounded: on a time-out the CTA raises kStatusWaitTimeout and runs through
// the remaining phases without waiting, so the kernel always ends.
#pragma once

#include "common.cuh"
#include "gemm_tc.cuh"      // mbarrier helpers, gelu_fast
#include "mixer.cuh"        // row_stats, norm4
#include "mixer_stream.cuh" // bulk_g2s
#include "select.cuh"       // SelectOut, write_token

namespace srm {
namespace sb {

constexpr int kThreads = 256, kWarps = 8;
constexpr int kMaxRows = 64;                 // samples per launch
constexpr int kPadBytes = 16;                // row padding in shared memory: ldmatrix rows land in distinct banks
constexpr int kLmChunkCols = 16;             // LM-head weight rows per pipeline stage
constexpr int kSmemBytes = 220 * 1024;
constexpr long long kBarrierLimitCycles = 1ll << 27;

struct LayerW {
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b, *alpha, *beta, *lam, *b1, *b2;
  const bf16 *W1, *W2;
};

struct Params {
  int B, d, F, V, h, n_ctx, L, t;
  float eps;
  const int32_t* tok_in;       // [B]
  const bf16* E;               // [V, d]
  const bf16* W_lm;            // [V, d]
  const float *lnf_g, *lnf_b;
  LayerW layer0;               // tensors of layer 0; layer l lies layer_bytes further on (all layers have one layout)
  int64_t layer_bytes;
  void* S;                     // cache of layer 0; layer l at S + l * layer_stride (bytes)
  int64_t layer_stride;
  float* x;                    // [B, d] residual stream
  bf16* a;                     // [B, d] activations (GEMM input)
  bf16* H;                     // [B, F]
  float* part;                 // [ks][B, d] partial sums of the down projection
  float* logits;               // [B, V] or nullptr (then only the greedy selection leaves the kernel)
  unsigned long long* best;    // [gridDim][B] per-CTA (sortable logit, ~column) of the LM-head slab
  uint32_t* bar;               // grid barrier counter, zero on entry
  uint32_t* status;
  const int32_t* ctr;          // device-side step counters or nullptr
  int greedy;                  // select inside the kernel
  SelectOut out;
  // slab plan (host): columns per CTA and CTAs used, per projection
  int up_cols, up_ctas;        // multiple of 8
  int dn_cols, dn_nslabs, dn_kslabs, dn_klen;   // dn_cols = 64; k-slab length a multiple of 16
  int lm_cols, lm_ctas;        // multiple of kLmChunkCols
};

__device__ __forceinline__ LayerW layer_w(const Params& p, int l) {
  const int64_t o = (int64_t)l * p.layer_bytes;
  auto f = [o](const float* q) { return reinterpret_cast<const float*>(reinterpret_cast<const uint8_t*>(q) + o); };
  auto b = [o](const bf16* q) { return reinterpret_cast<const bf16*>(reinterpret_cast<const uint8_t*>(q) + o); };
  const LayerW& w = p.layer0;
  return LayerW{f(w.ln1_g), f(w.ln1_b), f(w.ln2_g), f(w.ln2_b), f(w.alpha), f(w.beta), f(w.lam), f(w.b1), f(w.b2), b(w.W1), b(w.W2)};
}

// ---- grid-wide barrier ------------------------------------------------------------------------
// Arrive / wait on a monotonically increasing counter: barrier number n (1, 2, ...) is passed when the counter
// has reached n * gridDim.x. All CTAs are resident (cooperative launch), so the wait ends; it is bounded anyway.
struct GridBarrier {
  uint32_t* ctr;
  uint32_t n;          // barriers passed so far
  bool dead;           // a wait timed out: stop waiting (the same value in every thread of the CTA)
  uint32_t* status;
  int* shared_dead;    // a word of shared memory through which thread 0 tells the others
  __device__ void sync() {
    // what this CTA wrote is read after the barrier by other CTAs, partly by bulk copies (the async proxy)
    __threadfence();
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __syncthreads();
    ++n;
    if (threadIdx.x == 0) {
      __threadfence();
      atomicAdd(ctr, 1u);
      if (!dead) {
        const uint32_t want = n * gridDim.x;
        const long long t0 = clock64();
        while (*reinterpret_cast<volatile uint32_t*>(ctr) < want) {
          __nanosleep(64);
          if (clock64() - t0 > kBarrierLimitCycles) { dead = true; raise_status(status, kStatusWaitTimeout); break; }
        }
        __threadfence();
      }
      *shared_dead = dead ? 1 : 0;
    }
    __syncthreads();
    dead = *shared_dead != 0;
    asm volatile("fence.proxy.async.global;" ::: "memory");
  }
};

// ---- mma.sync m16n8k16 (bf16 x bf16 -> fp32) and its shared-memory fragment loads ----------------
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t (&r)[2], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// One 16 x 16 output tile over K (a multiple of 32): rows m0.. of A (row-major, lda bytes per row) times rows
// n0 .. n0 + 15 of W (row-major [n][k], ldw bytes per row), both in shared memory. c0 holds columns n0 .. n0 + 7, c1
// columns n0 + 8 .. n0 + 15; fragment layout: lane l holds c[0], c[1] = (row m0 + l / 4, columns 2 (l % 4), + 1 of its
// eight) and c[2], c[3] = the same columns of row + 8. Even and odd k-steps accumulate separately (four independent
// chains of dependent mma instructions instead of one: with a few rows the tile is latency-bound) and are added at
// the end.
__device__ __forceinline__ void tile_16x16(float (&c0)[4], float (&c1)[4], const uint8_t* A, int lda, int m0, const uint8_t* W,
                                           int ldw, int n0, int K, int lane) {
  float e0[4] = {0.f, 0.f, 0.f, 0.f}, e1[4] = {0.f, 0.f, 0.f, 0.f}, o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
  // A: matrices (rows 0-7, k 0-7), (rows 8-15, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15): lane l points at
  // row (l % 16), k offset 8 (l / 16). W: (n 0-7, k 0-7), (n 0-7, k 8-15), (n 8-15, k 0-7), (n 8-15, k 8-15): lane l
  // points at row (l % 8) + 8 (l / 16), k offset 8 ((l / 8) % 2).
  const uint32_t a_addr = tc::smem_u32(A + (size_t)(m0 + (lane & 15)) * lda + (lane >> 4) * 16);
  const uint32_t b_addr = tc::smem_u32(W + (size_t)(n0 + (lane & 7) + ((lane >> 4) << 3)) * ldw + ((lane >> 3) & 1) * 16);
#pragma unroll 2
  for (int k = 0; k < K; k += 32) {
    uint32_t a[4], b[4], a2[4], b2[4];
    ldsm_x4(a, a_addr + k * 2);
    ldsm_x4(b, b_addr + k * 2);
    ldsm_x4(a2, a_addr + k * 2 + 32);
    ldsm_x4(b2, b_addr + k * 2 + 32);
    const uint32_t bl[2] = {b[0], b[1]}, bh[2] = {b[2], b[3]}, bl2[2] = {b2[0], b2[1]}, bh2[2] = {b2[2], b2[3]};
    mma_bf16(e0, a, bl);
    mma_bf16(e1, a, bh);
    mma_bf16(o0, a2, bl2);
    mma_bf16(o1, a2, bh2);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) { c0[i] = e0[i] + o0[i]; c1[i] = e1[i] + o1[i]; }
}

// ---- shared-memory staging --------------------------------------------------------------------
// `rows` rows of `row_bytes` bytes (a multiple of 16), `src_stride` bytes apart in global memory, to rows
// `row_bytes + kPadBytes` apart in shared memory; completion is counted on `bar`. Called by all lanes of warp 0:
// lane 0 announces the bytes, then the lanes issue one bulk copy per row.
__device__ __forceinline__ void stage_rows(uint8_t* dst, const void* src, int rows, int row_bytes, int64_t src_stride,
                                           uint64_t* bar, int lane) {
  tc::fence_async_smem();          // earlier reads of the region (ordered by a barrier) come before the copies into it
  if (lane == 0) tc::mbar_expect_tx(bar, (uint32_t)rows * (uint32_t)row_bytes);
  __syncwarp();
  const uint8_t* s = static_cast<const uint8_t*>(src);
  for (int r = lane; r < rows; r += 32)
    bulk_g2s(dst + (size_t)r * (row_bytes + kPadBytes), s + (int64_t)r * src_stride, (uint32_t)row_bytes, bar);
}

// Bounded wait on a phase of `bar`; all threads of the CTA call it. False after a time-out.
__device__ __forceinline__ bool wait_stage(uint64_t* bar, uint32_t parity, uint32_t* status, bool dead) {
  if (dead) return false;
  return tc::mbar_wait(bar, parity, status);
}

// ---- row phase: one CTA per sample row -------------------------------------------------------------
// Sum over the CTA of one value per thread (all threads call it; `red` holds one float per warp).
__device__ __forceinline__ float cta_sum(float v, float* red) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) t += red[w];
  __syncthreads();                         // red may be written again
  return t;
}

// x_in = E[tok] (layer 0) or x + b2 of the previous layer + the partial sums of its down projection in slab order.
// layer < L: the fused mixer step (LN1, Eq. 2 / Eq. 3 update of the cache, residual, LN2), leaving x and the
// activation a. layer == L: a = LN_f(x_in). Thread i owns channels 4 i .. 4 i + 3 (d <= 1024): every global load
// of the row is issued before the first reduction, so the phase costs a few memory latencies, not one per vector.
template <typename ST>
__device__ __forceinline__ void row_phase(const Params& p, int layer, int64_t row, int t, float* red) {
  const int d = p.d, c = threadIdx.x * 4;
  const bool on = c < d;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 v = zero;
  if (layer == 0) {
    int tk = p.tok_in[row];
    if (tk < 0 || tk >= p.V) {
      if (threadIdx.x == 0) raise_status(p.status, kStatusTokenRange);
      tk = tk < 0 ? 0 : p.V - 1;
    }
    if (on) v = ldg4(p.E + (int64_t)tk * d + c);
  } else if (on) {
    // written by other CTAs in this kernel: not through L1
    float4 q[8];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      q[ks] = ks < p.dn_kslabs ? __ldcg(reinterpret_cast<const float4*>(p.part + ((int64_t)ks * p.B + row) * d + c)) : zero;
    v = __ldcg(reinterpret_cast<const float4*>(p.x + row * d + c));
    const float4 bb = ldg4(layer_w(p, layer - 1).b2 + c);
    v = make_float4(v.x + bb.x, v.y + bb.y, v.z + bb.z, v.w + bb.w);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) v = make_float4(v.x + q[ks].x, v.y + q[ks].y, v.z + q[ks].z, v.w + q[ks].w);
  }
  const bool last = layer == p.L;
  const LayerW w = layer_w(p, last ? 0 : layer);
  // parameters and the cache row: independent of the statistics, so their loads overlap the reductions
  float4 g1 = zero, b1 = zero, g2 = zero, b2n = zero, bt = zero, s = zero;
  float al = 0.f, lm = 0.f;
  int g = 0;
  ST* Sr = nullptr;
  if (on) {
    if (last) {
      g2 = ldg4(p.lnf_g + c); b2n = ldg4(p.lnf_b + c);
    } else {
      g = c / (d / p.h);
      g1 = ldg4(w.ln1_g + c); b1 = ldg4(w.ln1_b + c); g2 = ldg4(w.ln2_g + c); b2n = ldg4(w.ln2_b + c);
      bt = ldg4(w.beta + (int64_t)t * d + c);
      al = __ldg(w.alpha + (int64_t)g * p.n_ctx + t); lm = __ldg(w.lam + g);
      Sr = reinterpret_cast<ST*>(static_cast<uint8_t*>(p.S) + (int64_t)layer * p.layer_stride) + row * d + c;
      s = ld4(Sr);
    }
  }
  const float inv_d = 1.0f / (float)d;
  if (!last) {
    const float mean = cta_sum((v.x + v.y) + (v.z + v.w), red) * inv_d;
    const float4 cd = on ? make_float4(v.x - mean, v.y - mean, v.z - mean, v.w - mean) : zero;
    const float rstd = rsqrtf(cta_sum((cd.x * cd.x + cd.y * cd.y) + (cd.z * cd.z + cd.w * cd.w), red) * inv_d + p.eps);
    if (on) {
      const float4 z = norm4(v, mean, rstd, g1, b1);
      float4 y, sn;
      if (g < (p.h >> 1)) {       // row-repeat head, Eq. 2: y = a z + b + S ; S' = l (S + a z)
        const float4 u = make_float4(al * z.x, al * z.y, al * z.z, al * z.w);
        y = make_float4(u.x + bt.x + s.x, u.y + bt.y + s.y, u.z + bt.z + s.z, u.w + bt.w + s.w);
        sn = make_float4(lm * (s.x + u.x), lm * (s.y + u.y), lm * (s.z + u.z), lm * (s.w + u.w));
      } else {                    // column-repeat head, Eq. 3: y = a (z + S) + b ; S' = l (z + S)
        const float4 q = make_float4(z.x + s.x, z.y + s.y, z.z + s.z, z.w + s.w);
        y = make_float4(al * q.x + bt.x, al * q.y + bt.y, al * q.z + bt.z, al * q.w + bt.w);
        sn = make_float4(lm * q.x, lm * q.y, lm * q.z, lm * q.w);
      }
      st4(Sr, sn);
      v = make_float4(v.x + y.x, v.y + y.y, v.z + y.z, v.w + y.w);
      st4(p.x + row * d + c, v);
    }
  }
  const float mean = cta_sum((v.x + v.y) + (v.z + v.w), red) * inv_d;
  const float4 cd = on ? make_float4(v.x - mean, v.y - mean, v.z - mean, v.w - mean) : zero;
  const float rstd = rsqrtf(cta_sum((cd.x * cd.x + cd.y * cd.y) + (cd.z * cd.z + cd.w * cd.w), red) * inv_d + p.eps);
  if (on) st4(p.a + row * d + c, norm4(v, mean, rstd, g2, b2n));
}

// Shared memory: 128 bytes of mbarriers | activation rows (kMaxRows padded rows) | weight rows.
__host__ __device__ inline int act_region_bytes(int d, int klen) {
  const int k = d > klen ? d : klen;
  return (kMaxRows * (2 * k + kPadBytes) + 127) / 128 * 128;
}
__host__ __device__ inline int weight_region_bytes(int d, int up_cols, int dn_cols, int klen) {
  int b = up_cols * (2 * d + kPadBytes);
  const int dn = dn_cols * (2 * klen + kPadBytes), lm = 2 * kLmChunkCols * (2 * d + kPadBytes) + 4096;   // + partial sums
  b = b > dn ? b : dn;
  return b > lm ? b : lm;
}

__device__ __forceinline__ unsigned long long pack_best(float v, int col) {
  return ((unsigned long long)order_key(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)col);
}

template <typename ST>
__global__ void __launch_bounds__(kThreads, 1) step_small_kernel(const Params p) {
  extern __shared__ __align__(128) uint8_t sm[];
  uint64_t* barA = reinterpret_cast<uint64_t*>(sm);
  uint64_t* barW = barA + 1;                             // two stages
  float* red32 = reinterpret_cast<float*>(sm + 96);     // one float per warp for the row-phase reductions
  uint8_t* sA = sm + 128;
  uint8_t* sW = sA + act_region_bytes(p.d, p.dn_klen);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  const int d = p.d, F = p.F, B = p.B;
  if (threadIdx.x == 0) {
    tc::mbar_init(barA, 1); tc::mbar_init(&barW[0], 1); tc::mbar_init(&barW[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  uint32_t parA = 0, parW0 = 0, parW1 = 0;
  GridBarrier gb{p.bar, 0u, false, p.status, reinterpret_cast<int*>(sm + 64)};
  const int t = p.ctr != nullptr ? p.ctr[kCtrPos] : p.t;
  const int m_tiles = (B + 15) >> 4;
  const int ld_d = 2 * d + kPadBytes;

  // this CTA's slabs
  const bool up_on = cta < p.up_ctas;
  const int up_n0 = cta * p.up_cols;
  const int up_n = up_on ? (F - up_n0 < p.up_cols ? F - up_n0 : p.up_cols) : 0;
  const bool dn_on = cta < p.dn_nslabs * p.dn_kslabs;
  const int dn_ns = cta % p.dn_nslabs, dn_ks = cta / p.dn_nslabs;
  const int dn_k0 = dn_ks * p.dn_klen;
  const int dn_k = dn_on ? (F - dn_k0 < p.dn_klen ? F - dn_k0 : p.dn_klen) : 0;
  const int ld_k = 2 * dn_k + kPadBytes;
  const bool lm_on = cta < p.lm_ctas;
  const int lm_n0 = cta * p.lm_cols;
  const int lm_n = lm_on ? (p.V - lm_n0 < p.lm_cols ? p.V - lm_n0 : p.lm_cols) : 0;
  const int lm_chunks = (lm_n + kLmChunkCols - 1) / kLmChunkCols;
  const int lm_stage = kLmChunkCols * ld_d;

  auto stage_up = [&](int l) {            // warp 0: W1 rows of this CTA's columns
    if (up_on && warp == 0) stage_rows(sW, layer_w(p, l).W1 + (int64_t)up_n0 * d, up_n, 2 * d, 2 * (int64_t)d, &barW[0], lane);
  };
  auto stage_dn = [&](int l) {            // warp 0: W2 rows of the n-slab, columns of the k-slab
    if (dn_on && warp == 0)
      stage_rows(sW, layer_w(p, l).W2 + (int64_t)dn_ns * p.dn_cols * F + dn_k0, p.dn_cols, 2 * dn_k, 2 * (int64_t)F, &barW[0], lane);
  };
  auto stage_lm = [&](int ch) {           // warp 0: one chunk of LM-head rows into stage ch % 2
    if (lm_on && warp == 0 && ch < lm_chunks) {
      const int rows = lm_n - ch * kLmChunkCols < kLmChunkCols ? lm_n - ch * kLmChunkCols : kLmChunkCols;
      stage_rows(sW + (ch & 1) * lm_stage, p.W_lm + (int64_t)(lm_n0 + ch * kLmChunkCols) * d, rows, 2 * d, 2 * (int64_t)d,
                 &barW[ch & 1], lane);
    }
  };

  stage_up(0);
  for (int l = 0; l < p.L; ++l) {
    // ---- token mixer: one warp per row ----
    for (int64_t r = cta; r < B; r += G) row_phase<ST>(p, l, r, t, red32);
    gb.sync();

    // ---- up projection: H[:, slab] = gelu(a W1[slab]^T + b1) ----
    if (up_on) {
      if (warp == 0) stage_rows(sA, p.a, B, 2 * d, 2 * (int64_t)d, barA, lane);
      bool ok = wait_stage(barA, parA, p.status, gb.dead);
      ok = wait_stage(&barW[0], parW0, p.status, gb.dead) && ok;
      parA ^= 1u; parW0 ^= 1u;
      if (!ok) gb.dead = true;
      const float* b1 = layer_w(p, l).b1;
      const int n16 = (up_n + 15) >> 4, tiles = m_tiles * n16;
      for (int tile = warp; ok && tile < tiles; tile += kWarps) {
        const int mt = tile % m_tiles, nt = tile / m_tiles;
        float c0[4], c1[4];
        tile_16x16(c0, c1, sA, ld_d, mt * 16, sW, ld_d, nt * 16, d, lane);
        const int r0 = mt * 16 + (lane >> 2);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float (&c)[4] = hf ? c1 : c0;
          const int cl = nt * 16 + hf * 8 + 2 * (lane & 3);          // column inside the slab
          if (cl < up_n) {
            const int col = up_n0 + cl;
            const float2 bb = __ldg(reinterpret_cast<const float2*>(b1 + col));
            if (r0 < B)
              *reinterpret_cast<__nv_bfloat162*>(p.H + (int64_t)r0 * F + col) =
                  __floats2bfloat162_rn(tc::gelu_fast(c[0] + bb.x), tc::gelu_fast(c[1] + bb.y));
            if (r0 + 8 < B)
              *reinterpret_cast<__nv_bfloat162*>(p.H + (int64_t)(r0 + 8) * F + col) =
                  __floats2bfloat162_rn(tc::gelu_fast(c[2] + bb.x), tc::gelu_fast(c[3] + bb.y));
          }
        }
      }
    }
    __syncthreads();                       // the weight rows have been read: the region may be refilled
    stage_dn(l);
    gb.sync();

    // ---- down projection: part[ks][:, n-slab] = H[:, k-slab] W2[n-slab, k-slab]^T ----
    if (dn_on) {
      if (warp == 0) stage_rows(sA, p.H + dn_k0, B, 2 * dn_k, 2 * (int64_t)F, barA, lane);
      bool ok = wait_stage(barA, parA, p.status, gb.dead);
      ok = wait_stage(&barW[0], parW0, p.status, gb.dead) && ok;
      parA ^= 1u; parW0 ^= 1u;
      if (!ok) gb.dead = true;
      float* out = p.part + (int64_t)dn_ks * B * d;
      const int tiles = m_tiles * (p.dn_cols >> 4);
      for (int tile = warp; ok && tile < tiles; tile += kWarps) {
        const int mt = tile % m_tiles, nt = tile / m_tiles;
        float c0[4], c1[4];
        tile_16x16(c0, c1, sA, ld_k, mt * 16, sW, ld_k, nt * 16, dn_k, lane);
        const int col = dn_ns * p.dn_cols + nt * 16 + 2 * (lane & 3), r0 = mt * 16 + (lane >> 2);
        if (r0 < B) {
          *reinterpret_cast<float2*>(out + (int64_t)r0 * d + col) = make_float2(c0[0], c0[1]);
          *reinterpret_cast<float2*>(out + (int64_t)r0 * d + col + 8) = make_float2(c1[0], c1[1]);
        }
        if (r0 + 8 < B) {
          *reinterpret_cast<float2*>(out + (int64_t)(r0 + 8) * d + col) = make_float2(c0[2], c0[3]);
          *reinterpret_cast<float2*>(out + (int64_t)(r0 + 8) * d + col + 8) = make_float2(c1[2], c1[3]);
        }
      }
    }
    __syncthreads();
    if (l + 1 < p.L) stage_up(l + 1);
    else { stage_lm(0); stage_lm(1); }
    gb.sync();
  }

  // ---- final norm ----
  for (int64_t r = cta; r < B; r += G) row_phase<ST>(p, p.L, r, t, red32);
  gb.sync();

  // ---- LM head over this CTA's vocabulary slab, chunk by chunk through two stages ----
  if (lm_on) {
    if (warp == 0) stage_rows(sA, p.a, B, 2 * d, 2 * (int64_t)d, barA, lane);
    bool ok = wait_stage(barA, parA, p.status, gb.dead);
    parA ^= 1u;
    // Every chunk is one 16-column tile per 16 rows. Warp w takes row tile w % 4 and half w / 4 of K; the upper
    // halves' partial sums go through shared memory to the lower warps, which own the results.
    const int mt = warp & 3, kh = warp >> 2;
    const int k_half = d >> 1;
    float* xch = reinterpret_cast<float*>(sW + 2 * lm_stage);   // [4 row tiles][32 lanes][8] partial sums
    float bv0 = -INFINITY, bv1 = -INFINITY;
    int bi0 = 0x7fffffff, bi1 = 0x7fffffff;
    bool bad = false;
    for (int ch = 0; ch < lm_chunks; ++ch) {
      const int s = ch & 1;
      ok = wait_stage(&barW[s], s ? parW1 : parW0, p.status, gb.dead || !ok) && ok;
      if (s) parW1 ^= 1u; else parW0 ^= 1u;
      const int rows = lm_n - ch * kLmChunkCols < kLmChunkCols ? lm_n - ch * kLmChunkCols : kLmChunkCols;
      float c0[4], c1[4];
      const bool work = ok && mt < m_tiles;
      if (work) {
        tile_16x16(c0, c1, sA + kh * k_half * 2, ld_d, mt * 16, sW + s * lm_stage + kh * k_half * 2, ld_d, 0, k_half, lane);
        if (kh == 1) {
          float4* o = reinterpret_cast<float4*>(xch + (mt * 32 + lane) * 8);
          o[0] = make_float4(c0[0], c0[1], c0[2], c0[3]);
          o[1] = make_float4(c1[0], c1[1], c1[2], c1[3]);
        }
      }
      __syncthreads();                                           // partial sums are visible; stage s has been read
      stage_lm(ch + 2);
      if (work && kh == 0) {
        const float4* o = reinterpret_cast<const float4*>(xch + (mt * 32 + lane) * 8);
        const float4 q0 = o[0], q1 = o[1];
        c0[0] += q0.x; c0[1] += q0.y; c0[2] += q0.z; c0[3] += q0.w;
        c1[0] += q1.x; c1[1] += q1.y; c1[2] += q1.z; c1[3] += q1.w;
        const int col = lm_n0 + ch * kLmChunkCols + 2 * (lane & 3), r0 = mt * 16 + (lane >> 2);
        const bool second = rows > 8;                            // V is a multiple of 8: a last chunk may hold 8 columns
        if (p.logits != nullptr) {
          if (r0 < B) {
            *reinterpret_cast<float2*>(p.logits + (int64_t)r0 * p.V + col) = make_float2(c0[0], c0[1]);
            if (second) *reinterpret_cast<float2*>(p.logits + (int64_t)r0 * p.V + col + 8) = make_float2(c1[0], c1[1]);
          }
          if (r0 + 8 < B) {
            *reinterpret_cast<float2*>(p.logits + (int64_t)(r0 + 8) * p.V + col) = make_float2(c0[2], c0[3]);
            if (second) *reinterpret_cast<float2*>(p.logits + (int64_t)(r0 + 8) * p.V + col + 8) = make_float2(c1[2], c1[3]);
          }
        }
        // (rows past B of a partly filled tile hold whatever the shared memory held: not looked at)
        if (r0 < B) bad |= !(c0[0] == c0[0]) | !(c0[1] == c0[1]) | (second & (!(c1[0] == c1[0]) | !(c1[1] == c1[1])));
        if (r0 + 8 < B) bad |= !(c0[2] == c0[2]) | !(c0[3] == c0[3]) | (second & (!(c1[2] == c1[2]) | !(c1[3] == c1[3])));
        if (c0[0] > bv0) { bv0 = c0[0]; bi0 = col; }            // ascending columns: the lowest among equals is kept
        if (c0[1] > bv0) { bv0 = c0[1]; bi0 = col + 1; }
        if (c0[2] > bv1) { bv1 = c0[2]; bi1 = col; }
        if (c0[3] > bv1) { bv1 = c0[3]; bi1 = col + 1; }
        if (second) {
          if (c1[0] > bv0) { bv0 = c1[0]; bi0 = col + 8; }
          if (c1[1] > bv0) { bv0 = c1[1]; bi0 = col + 9; }
          if (c1[2] > bv1) { bv1 = c1[2]; bi1 = col + 8; }
          if (c1[3] > bv1) { bv1 = c1[3]; bi1 = col + 9; }
        }
      }
      __syncthreads();                                           // the partial sums have been taken
    }
    if (!ok) gb.dead = true;
    if (p.greedy) {
      // per row: over the four lanes of a quad (their columns interleave, so the packed (value, lowest column) decides)
      unsigned long long k0 = bi0 == 0x7fffffff ? 0ull : pack_best(bv0, bi0), k1 = bi1 == 0x7fffffff ? 0ull : pack_best(bv1, bi1);
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {
        const unsigned long long q0 = __shfl_xor_sync(0xffffffffu, k0, o), q1 = __shfl_xor_sync(0xffffffffu, k1, o);
        k0 = q0 > k0 ? q0 : k0; k1 = q1 > k1 ? q1 : k1;
      }
      unsigned long long* red = reinterpret_cast<unsigned long long*>(sW);      // the weight stages are free now
      if (kh == 0 && (lane & 3) == 0) { red[mt * 16 + (lane >> 2)] = k0; red[mt * 16 + 8 + (lane >> 2)] = k1; }
      __syncthreads();
      if (threadIdx.x < B) p.best[(int64_t)cta * B + threadIdx.x] = red[threadIdx.x];
      if (bad) raise_status(p.status, kStatusNonFinite);
    }
  }
  if (!p.greedy) return;                   // the caller selects from the logits
  gb.sync();
  if (cta == 0 && threadIdx.x < B) {
    unsigned long long best = 0ull;
    for (int c = 0; c < p.lm_ctas; ++c) {
      const unsigned long long k = __ldcg(p.best + (int64_t)c * B + threadIdx.x);
      best = k > best ? k : best;
    }
    int tok = best == 0ull ? 0 : (int)(0xFFFFFFFFu - (uint32_t)(best & 0xFFFFFFFFull));
    if (tok < 0 || tok >= p.V) tok = 0;
    write_token(p.out, threadIdx.x, tok);
  }
}

}  // namespace sb
}  // namespace srm
