// bf16 projection D[M,N] = A[M,K] * W[N,K]^T on the 5th-generation tensor cores (sm_100a).
//
// Two CTAs of a cluster (a CTA pair on neighbouring SMs) own one 256 x 256 output tile:
//   TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast): CTA r loads rows
//   [128 r, 128 r + 128) of the A tile and of the W tile into its own shared-memory ring;
//   both CTAs' copies complete on the leader CTA's mbarrier;
//   tcgen05.mma.cta_group::2 (one issuing thread in the leader CTA, 256x256x16 per instruction)
//   reads both CTAs' shared memory and accumulates in fp32 in both CTAs' tensor memory (each holds
//   its 128 rows x 256 columns, two such buffers, so the epilogue of tile i overlaps the main loop
//   of tile i+1); tcgen05.commit multicasts "stage free" / "accumulator ready" to both CTAs;
//   tcgen05.ld -> fused epilogue -> global memory, in each CTA for its own 128 rows.
// Pairing halves the W bytes each SM pulls from L2 per flop compared with a 128 x 256 tile per
// SM, which is what bounded the single-CTA version of this kernel.
//
// The kernel is persistent: grid = 2 * min(pieces, resident clusters), pieces taken round-robin; a piece is a
// whole tile or, for the tiles of a partly filled last round, one of its two 256 x 128 halves (GemmArgs::tail_tiles).
// Warp roles per CTA: warp 0 = TMA producer, warp 1 = MMA issuer (leader only) and TMEM owner,
// warps 2..17 = epilogue (warp w reads TMEM lanes 32*(w%4) .. +31, one accumulator row per thread;
// the four warps that share a lane quarter split the tile's columns; four warps per scheduler hide
// each other's TMEM / shared / global latencies, since with K = d the epilogue's instruction issue
// is as long as the tile's MMAs). Each epilogue warp stages 32 rows x 128 bytes of finished
// output in a private, 128-byte-swizzled shared-memory buffer and hands it to the TMA unit: a tiled
// bulk store for the activation and logit epilogues, a tiled bulk reduce-add (fp32 add performed in
// L2) for the residual epilogue, so no thread computes a global address, waits on a global load of
// x, or holds a store in flight. Every element of x receives exactly one add per launch, so the
// result does not depend on timing. Rows and columns beyond M, N are clipped by the TMA unit.
// Every wait is bounded: after ~2^31 clock cycles a waiter raises kStatusWaitTimeout, leaves its
// loop, and both CTAs still meet at the final cluster barrier, release tensor memory and exit.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "gemm_simt.cuh"   // GemmEpilogue enum

namespace srm {
namespace tc {

constexpr int BM = 256, BN = 256, BK = 64;       // tile of one CTA pair
constexpr int kRowsPerCta = 128;                 // A rows and W rows each CTA loads per k-block
constexpr int kStages = 5;
constexpr int kAStageBytes = kRowsPerCta * BK * 2;   // 16 KiB
constexpr int kBStageBytes = kRowsPerCta * BK * 2;   // 16 KiB
constexpr int kStageBytes = kAStageBytes + kBStageBytes;
constexpr int kBarrierBytes = 256;
constexpr int kEpiWarps = 16;
constexpr int kColsPerEpiWarp = BN / (kEpiWarps / 4);   // 64
constexpr int kOutBoxRows = 32;                  // one epilogue warp's rows
constexpr int kOutBoxBytes = kOutBoxRows * 128;  // staging buffer of one epilogue warp: 32 rows x 128 bytes
constexpr int kSmemBytes = kStages * kStageBytes + kEpiWarps * kOutBoxBytes + kBarrierBytes + 1024;  // +1024: alignment
constexpr int kThreads = 64 + kEpiWarps * 32;
constexpr int kTmemCols = 512;                   // two accumulators of BN fp32 columns
constexpr long long kWaitLimitCycles = 1ll << 31;

// ---- raw PTX wrappers ---------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One try: the thread may be suspended by the hardware until the phase completes or the hint (nanoseconds) has
// passed. With the hint a waiting warp stays off the issue ports instead of re-trying at once: under the power
// cap that is worth 120 MHz of SM clock to the decode step (1.50 -> 1.47 ms), most of it in the LM head, whose 16
// epilogue warps per CTA wait for an accumulator most of the time.
constexpr uint32_t kTryWaitHintNs = 1000;
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kTryWaitHintNs)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false (after raising the status bit) when the phase has not completed within `limit` clock
// cycles (the pipelines use kWaitLimitCycles: far longer than any kernel of this library runs).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* status,
                                          long long limit = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) {
      raise_status(status, kStatusWaitTimeout);
      return false;
    }
  }
}

// One thread waits, with the bounded wait every pipeline of this library uses, on an mbarrier phase that nothing
// ever completes: the wait must give up after `limit` cycles, raise kStatusWaitTimeout and let the kernel end.
// (The host-visible check that a stuck pipeline cannot hang the GPU.)
__global__ void wait_probe_kernel(uint32_t* status, long long limit, int* gave_up) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(&bar, 0u, status, limit);
    if (gave_up != nullptr) *gave_up = ok ? 0 : 1;
  }
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t mapa(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive (optionally announcing transaction bytes) on an mbarrier anywhere in the cluster
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load into this CTA's shared memory whose completion is counted on an mbarrier that may
// live in the peer CTA of the pair (cta_group::2); no multicast.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on the mbarrier at this shared-memory offset in BOTH CTAs of the pair once all tcgen05
// operations issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask)
               : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- bulk tensor stores (shared -> global), tracked per issuing thread in bulk async-groups ----
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(x), "r"(y)
               : "memory");
}
// Same store, marked evict-first in L2: for output that is written once and not read again soon (the
// logits), so that it does not push the operands the mainloop keeps re-reading out of L2.
__device__ __forceinline__ void tma_store_2d_streaming(const CUtensorMap* map, const void* src, int x, int y) {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(x), "r"(y), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, const void* src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the bulk operations committed by this thread have finished READING shared memory
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... have completed altogether
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// orders this thread's generic-proxy writes to shared memory before later async-proxy (TMA) reads
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements)
// laid out by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes apart (SBO), the
// leading-dimension offset is not used by swizzled K-major layouts, descriptor version 1,
// layout type 2 (SWIZZLE_128B). Stepping 16 elements along K adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = BN, M = BM (pair).
__host__ __device__ constexpr uint32_t instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(BM >> 4) << 24);
}
constexpr uint32_t kInstrDesc = instr_desc(BN);
constexpr int kHalfN = BN / 2;                   // width of the pieces the last tiles may be cut into

struct GemmArgs {
  int64_t M, N, K;
  const float* bias;   // [N] (epilogues 0, 1)
  void* out;           // bf16 [M,N] (epilogue 0), float [M,N] (epilogues 1, 2), or for kEpiArgmax the partial
                       // results uint2 [argmax_slots(N)][M] = (bits of the slice maximum, its column)
  uint32_t* status;
  int w_static;        // W is constant data (model weights): its first tiles may be fetched before pdl_wait()
  // kEpiCollect: out = candidate lists, unsigned long long [M][cap]; an element v of row r in column c with
  // v >= thr[r] takes the next free place of row r (cnt[r], counted atomically; places beyond cap are dropped but
  // counted) as ((~order_key(v)) << 32 | c): ascending order of these words is (value descending, column ascending).
  const float* thr;    // [M] per-row thresholds; a NaN or all-zero word means "none": nothing is collected
  uint32_t* cnt;       // [M] zero on entry
  int cap;
  // Only the first *m_limit rows (a device word written by an earlier kernel of the stream) are computed; nullptr:
  // all M rows. The first weight tiles are then not fetched ahead of the dependency wait.
  const uint32_t* m_limit;
  // The last `tail_tiles` tiles (in tile order) are processed as two pieces of 128 columns each, so that a last,
  // partly filled round of tiles keeps (nearly) all CTA pairs busy: a half piece moves three quarters of a tile's
  // operand bytes for half its flops, and 2 r half pieces on 74 pairs end earlier than r tiles on r pairs.
  int tail_tiles;
  // kEpiPlain only. k_slices > 1: the K dimension of every tile is cut into k_slices equal ranges of k-blocks, a
  // piece is (tile, range), and range s writes its partial product to rows [s * plane_rows, s * plane_rows + M) of
  // the output (plane_rows a multiple of 256, >= M): with a few tiles and a long K (the down projection of a small
  // batch: 4 tiles of 64 k-blocks for 74 pairs) all pairs work on it, and the consumer adds the planes in a fixed
  // order. No half-width pieces then.
  int k_slices;
  int64_t plane_rows;
};

// Piece q of a launch: the tile it belongs to, its first column inside the tile and its width.
struct Piece { int64_t tile; int noff, nw; };
__device__ __forceinline__ Piece piece_of(int64_t q, int64_t tiles, int tail) {
  const int64_t whole = tiles - tail;
  if (q < whole) return Piece{q, 0, BN};
  const int64_t j = q - whole;
  return Piece{whole + (j >> 1), (int)(j & 1) * kHalfN, kHalfN};
}

// order-preserving map float -> uint32 (larger float, larger key)
__device__ __forceinline__ uint32_t order_key_bits(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// kEpiArgmax: one partial result per row and per 64-column slice of the (256-column padded) output.
__host__ __device__ inline int64_t argmax_slots(int64_t N) { return (N + BN - 1) / BN * (BN / 64); }

// GELU(v) = v * Phi(v) with the normal CDF written as a logistic function of an odd polynomial,
//   Phi(v) ~= 1 / (1 + exp(-v (a + b v^2 + c v^4))),   a = 1.59501055, b = 7.40160400e-2, c = -7.03804784e-4
// (coefficients fitted to minimise the maximum error of v * Phi(v) over the real line: 2.6e-5), evaluated
// through 1 / (1 + exp(-w)) = (1 + tanh(w / 2)) / 2 with the hardware tanh (absolute error below 2^-10.9),
// so |error| <= 2.6e-5 + |v| / 2 * 5.2e-4: below a quarter of the bf16 spacing of the hidden activation it
// produces. v^2 is clamped at 64 so the polynomial stays positive; beyond |v| = 8 tanh is +-1 anyway.
// Eight instructions per element, one on the special-function unit: the epilogue shares the SM with the
// next tile's MMAs, and with erf, or with ex2 + rcp, the special-function unit alone took half a tile time.
__device__ __forceinline__ float tanh_approx(float x) {
  float r;
  asm("tanh.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float gelu_fast(float v) {
  const float s = fminf(v * v, 64.0f);
  float q = fmaf(s, -0.5f * 7.03804784e-4f, 0.5f * 7.40160400e-2f);
  q = fmaf(s, q, 0.5f * 1.59501055f);                    // (a + b s + c s^2) / 2
  const float t = tanh_approx(q * v);
  const float hv = 0.5f * v;
  return fmaf(hv, t, hv);
}

// Hands this warp's 32 rows x 128 bytes (v = the 32 words of the lane's row) to the TMA unit.
// The staging buffer uses the 128-byte swizzle of the output tensor map: the 16-byte piece q of row r
// sits at piece q ^ (r % 8), which also makes the eight lanes of a quarter-warp hit distinct banks.
// Lane 0 issues the bulk operation and is the only thread that tracks its completion.
template <int EPI>
__device__ __forceinline__ void emit_box(const CUtensorMap* tmD, uint8_t* buf, int lane, int col, int row,
                                         const uint32_t (&v)[32]) {
  if (lane == 0) bulk_wait_read();          // the previous box has left the buffer
  __syncwarp();
  uint8_t* mine = buf + lane * 128;
#pragma unroll
  for (int q = 0; q < 8; ++q)
    *reinterpret_cast<uint4*>(mine + ((q ^ (lane & 7)) << 4)) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
  fence_async_smem();
  __syncwarp();
  if (lane == 0) {
    if (EPI == kEpiBiasResidual) tma_reduce_add_2d(tmD, buf, col, row);
    else if (EPI == kEpiPlain) tma_store_2d_streaming(tmD, buf, col, row);
    else tma_store_2d(tmD, buf, col, row);
    bulk_commit();
  }
}

// max(a, b, c) that returns NaN when any input is NaN
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float r;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// Greedy selection over 16 consecutive logits r[0..15] of columns col .. col+15, folded into the running
// (bv, bi) with the rule of the stand-alone selection kernel: largest value, lowest column among equals,
// NaN never wins. The chunk maximum costs half an instruction per element; the column search runs only in
// lanes whose chunk beats their running maximum.
__device__ __forceinline__ void argmax_chunk16(const uint32_t (&r)[16], int col, int64_t N, float& bv, int& bi, bool& bad) {
  float f[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(r[j]);
  if (col + 16 <= N) {
    const float m = max3_nan(max3_nan(max3_nan(f[0], f[1], f[2]), max3_nan(f[3], f[4], f[5]), max3_nan(f[6], f[7], f[8])),
                             max3_nan(max3_nan(f[9], f[10], f[11]), max3_nan(f[12], f[13], f[14]), f[15]), -INFINITY);
    if (m == m) {                       // no NaN in the chunk
      if (m > bv) {
        int idx = 15;
#pragma unroll
        for (int j = 14; j >= 0; --j) idx = (f[j] == m) ? j : idx;
        bv = m;
        bi = col + idx;
      }
      return;
    }
  }
  // a NaN somewhere, or the ragged end of the row: the element-by-element rule
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    if (col + j < N) {
      bad |= !(f[j] == f[j]);
      if (f[j] > bv || (f[j] == bv && col + j < bi)) { bv = f[j]; bi = col + j; }
    }
  }
}

// Top-k candidates among 16 consecutive logits r[0..15] of columns col .. col+15 of this lane's row: everything
// at or above the row's threshold goes to the row's list. The chunk maximum decides in eight instructions
// whether the lane has anything to do (about one chunk in ten has, with some 200 candidates per row of 32000).
// A NaN never qualifies (it is reported through `bad`).
__device__ __forceinline__ void collect_chunk16(const uint32_t (&r)[16], int col, const GemmArgs& g, int64_t row, float thr,
                                                bool& bad) {
  float f[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(r[j]);
  const float m = max3_nan(max3_nan(max3_nan(f[0], f[1], f[2]), max3_nan(f[3], f[4], f[5]), max3_nan(f[6], f[7], f[8])),
                           max3_nan(max3_nan(f[9], f[10], f[11]), max3_nan(f[12], f[13], f[14]), f[15]), -INFINITY);
  if (m >= thr || m != m) {
    unsigned long long* list = reinterpret_cast<unsigned long long*>(g.out) + row * (int64_t)g.cap;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (col + j < g.N) {
        bad |= !(f[j] == f[j]);
        if (f[j] >= thr) {
          const uint32_t slot = atomicAdd(g.cnt + row, 1u);
          if (slot < (uint32_t)g.cap)
            list[slot] = ((unsigned long long)(~order_key_bits(f[j])) << 32) | (uint32_t)(col + j);
        }
      }
    }
  }
}

// The 64 accumulator columns [col0, col0 + 64) of this warp's 32 rows: TMEM -> registers -> bias /
// activation -> one (bf16) or two (fp32) boxes of 128 bytes per row, or the fused greedy selection.
// The columns come in four chunks of 16; the load of chunk i+1 is in flight while chunk i is processed
// (tcgen05.wait::ld waits for every load of the thread, so it is placed after the processing).
template <int EPI>
__device__ __forceinline__ void epilogue_columns(const GemmArgs& g, const CUtensorMap* tmD, uint8_t* buf, int lane,
                                                 uint32_t taddr, int row0, int col0) {
  constexpr int kChunks = kColsPerEpiWarp / 16;
  uint32_t ra[16], rb[16];
  uint32_t v[32];                        // staged output words of the lane's row (not used by kEpiArgmax)
  float bv = -INFINITY;                  // kEpiArgmax: running maximum and its column
  int bi = 0x7fffffff;
  bool bad = false;
  float thr = INFINITY;                  // kEpiCollect: this row's threshold
  if (EPI == kEpiCollect && row0 + lane < g.M) {
    thr = __ldg(g.thr + row0 + lane);
    if (!(thr == thr) || __float_as_uint(thr) == 0u) thr = INFINITY;
  }
  tmem_ld16(taddr, ra);
  tmem_ld_wait();
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    uint32_t (&cur)[16] = (c & 1) ? rb : ra;
    uint32_t (&nxt)[16] = (c & 1) ? ra : rb;
    if (c + 1 < kChunks) tmem_ld16(taddr + 16 * (c + 1), nxt);
    const int col = col0 + 16 * c;
    if (EPI == kEpiArgmax) {
      if (col < g.N) argmax_chunk16(cur, col, g.N, bv, bi, bad);
    } else if (EPI == kEpiCollect) {
      if (col < g.N && row0 + lane < g.M) collect_chunk16(cur, col, g, row0 + lane, thr, bad);
    } else if (EPI == kEpiBiasGelu) {
#pragma unroll
      for (int j = 0; j < 16; j += 4) {
        float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col + j < g.N) b = __ldg(reinterpret_cast<const float4*>(g.bias + col + j));
        __nv_bfloat162 p;
        p = __floats2bfloat162_rn(gelu_fast(__uint_as_float(cur[j + 0]) + b.x), gelu_fast(__uint_as_float(cur[j + 1]) + b.y));
        v[8 * c + j / 2] = *reinterpret_cast<uint32_t*>(&p);
        p = __floats2bfloat162_rn(gelu_fast(__uint_as_float(cur[j + 2]) + b.z), gelu_fast(__uint_as_float(cur[j + 3]) + b.w));
        v[8 * c + j / 2 + 1] = *reinterpret_cast<uint32_t*>(&p);
      }
      if (c == kChunks - 1) emit_box<EPI>(tmD, buf, lane, col0, row0, v);
    } else {
#pragma unroll
      for (int j = 0; j < 16; j += 4) {
        if (EPI == kEpiBiasResidual && g.bias != nullptr && col + j < g.N) {
          const float4 b = __ldg(reinterpret_cast<const float4*>(g.bias + col + j));
          v[16 * (c & 1) + j + 0] = __float_as_uint(__uint_as_float(cur[j + 0]) + b.x);
          v[16 * (c & 1) + j + 1] = __float_as_uint(__uint_as_float(cur[j + 1]) + b.y);
          v[16 * (c & 1) + j + 2] = __float_as_uint(__uint_as_float(cur[j + 2]) + b.z);
          v[16 * (c & 1) + j + 3] = __float_as_uint(__uint_as_float(cur[j + 3]) + b.w);
        } else {
          v[16 * (c & 1) + j + 0] = cur[j + 0]; v[16 * (c & 1) + j + 1] = cur[j + 1];
          v[16 * (c & 1) + j + 2] = cur[j + 2]; v[16 * (c & 1) + j + 3] = cur[j + 3];
        }
      }
      // two chunks make one box of 32 fp32 columns; a box that starts beyond N is not emitted
      if ((c & 1) && col - 16 < g.N) emit_box<EPI>(tmD, buf, lane, col - 16, row0, v);
    }
    if (c + 1 < kChunks) tmem_ld_wait();
  }
  if (EPI == kEpiCollect && bad) raise_status(g.status, kStatusNonFinite);
  if (EPI == kEpiArgmax) {
    if (bad) raise_status(g.status, kStatusNonFinite);
    const int64_t slot = col0 / kColsPerEpiWarp;
    const int64_t row = row0 + lane;
    if (row < g.M) reinterpret_cast<uint2*>(g.out)[slot * g.M + row] = make_uint2(__float_as_uint(bv), (uint32_t)bi);
  }
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmD, const __grid_constant__ CUtensorMap tmB64, const GemmArgs g) {
  pdl_trigger();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // The selecting epilogues stage nothing in shared memory: their 64 KB of output boxes become two more operand
  // stages (seven k-blocks in flight per SM instead of five).
  constexpr bool kNoBoxes = EPI == kEpiArgmax || EPI == kEpiCollect;
  constexpr int NS = kNoBoxes ? kStages + 2 : kStages;
  static_assert(NS * kStageBytes + (kNoBoxes ? 0 : kEpiWarps * kOutBoxBytes) + kBarrierBytes + 1024 <= kSmemBytes, "shared memory");
  uint8_t* sA = smem;
  uint8_t* sB = smem + NS * kAStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + NS * kStageBytes + (kNoBoxes ? 0 : kEpiWarps * kOutBoxBytes));   // used in the leader CTA
  uint64_t* empty = full + NS;           // per CTA: stage may be refilled
  uint64_t* tfull = empty + NS;     // per CTA [2]: accumulator ready for the epilogue
  uint64_t* tempty = tfull + 2;          // leader [2]: accumulator drained by both CTAs' epilogues
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  uint8_t* boxes = smem + NS * kStageBytes;           // 1024-byte aligned, one staging buffer per epilogue warp (not with kNoBoxes)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();           // 0 = leader of the pair
  const int64_t cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 2 * kEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  cluster_sync();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Barriers, tensor memory and the cluster handshake are set up; from here on global memory is touched.
  // The producer thread orders itself (it may fetch weights, which no kernel writes, ahead of the wait).
  if (threadIdx.x != 0 || g.m_limit != nullptr) pdl_wait();
  int64_t M_rows = g.M;
  if (g.m_limit != nullptr) {              // a row count left on the device by an earlier kernel
    const int64_t lim = (int64_t)*reinterpret_cast<const volatile uint32_t*>(g.m_limit);
    M_rows = lim < M_rows ? lim : M_rows;
  }

  const int64_t m_tiles = (M_rows + BM - 1) / BM, n_tiles = (g.N + BN - 1) / BN;
  const int64_t tiles = m_tiles * n_tiles;
  const int ks = (EPI == kEpiPlain && g.k_slices > 1 && g.m_limit == nullptr) ? g.k_slices : 1;   // ranges of K per tile
  const int tail = (g.m_limit != nullptr || ks > 1) ? 0 : g.tail_tiles;
  const int64_t pieces = (tiles + tail) * ks;          // a tail tile counts as two pieces
  const int k_all = static_cast<int>(g.K / BK);
  const int k_blocks = (k_all + ks - 1) / ks;          // k-blocks per piece (the last range of a tile may be shorter)

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // While the predecessor kernel drains: start the first tile's W loads (the ring is empty, so
      // the first NS stages need no wait), then order against the predecessor and add the A loads.
      int pre = 0;
      if (cluster_id < pieces) {
        const Piece pc = piece_of(cluster_id / ks, tiles, tail);
        const int kb0 = static_cast<int>(cluster_id % ks) * k_blocks;          // first k-block of this piece's range
        const int kbn = k_all - kb0 < k_blocks ? k_all - kb0 : k_blocks;
        const int w_rows = pc.nw >> 1;                                       // W rows each CTA of the pair loads
        const CUtensorMap* mapB = pc.nw == BN ? &tmB : &tmB64;
        const uint32_t stage_bytes = kAStageBytes + (uint32_t)w_rows * BK * 2;
        const int m0 = static_cast<int>(pc.tile % m_tiles) * BM + static_cast<int>(rank) * kRowsPerCta;
        const int n0 = static_cast<int>(pc.tile / m_tiles) * BN + pc.noff + static_cast<int>(rank) * w_rows;
        pre = kbn < NS ? (kbn > 0 ? kbn : 0) : NS;
        if (!g.w_static) pdl_wait();
        for (int kb = 0; kb < pre; ++kb) {
          const uint32_t full_leader = mapa(smem_u32(&full[kb]), 0);
          mbar_expect_tx_cluster(full_leader, stage_bytes);
          tma_load_2d(sB + kb * kBStageBytes, mapB, full_leader, (kb0 + kb) * BK, n0);
        }
        if (g.w_static) pdl_wait();
        for (int kb = 0; kb < pre; ++kb)
          tma_load_2d(sA + kb * kAStageBytes, &tmA, mapa(smem_u32(&full[kb]), 0), (kb0 + kb) * BK, m0);
        stage = pre;
        if (stage == NS) { stage = 0; phase ^= 1u; }
      } else {
        pdl_wait();
      }
      for (int64_t q = cluster_id; ok && q < pieces; q += n_clusters) {
        const Piece pc = piece_of(q / ks, tiles, tail);
        const int kb0 = static_cast<int>(q % ks) * k_blocks;
        const int kbn = k_all - kb0 < k_blocks ? k_all - kb0 : k_blocks;
        const int w_rows = pc.nw >> 1;
        const CUtensorMap* mapB = pc.nw == BN ? &tmB : &tmB64;
        const uint32_t stage_bytes = kAStageBytes + (uint32_t)w_rows * BK * 2;
        const int m0 = static_cast<int>(pc.tile % m_tiles) * BM + static_cast<int>(rank) * kRowsPerCta;
        const int n0 = static_cast<int>(pc.tile / m_tiles) * BN + pc.noff + static_cast<int>(rank) * w_rows;
        for (int kb = (q == cluster_id ? pre : 0); kb < kbn; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1u, g.status)) { ok = false; break; }
          const uint32_t full_leader = mapa(smem_u32(&full[stage]), 0);
          mbar_expect_tx_cluster(full_leader, stage_bytes);
          tma_load_2d(sA + stage * kAStageBytes, &tmA, full_leader, (kb0 + kb) * BK, m0);
          tma_load_2d(sB + stage * kBStageBytes, mapB, full_leader, (kb0 + kb) * BK, n0);
          if (++stage == NS) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // a consumer gave up: give the copies already issued time to land before the CTA can exit
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 21)) { }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (rank == 0 && lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int64_t q = cluster_id; ok && q < pieces; q += n_clusters) {
        const uint32_t idesc = instr_desc(piece_of(q / ks, tiles, tail).nw);
        const int kb0 = static_cast<int>(q % ks) * k_blocks;
        const int kbn = k_all - kb0 < k_blocks ? k_all - kb0 : k_blocks;
        if (!mbar_wait(&tempty[acc], acc_phase ^ 1u, g.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = 0; kb < kbn; ++kb) {
          if (!mbar_wait(&full[stage], phase, g.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = make_smem_desc(smem_u32(sA + stage * kAStageBytes));
          const uint64_t db = make_smem_desc(smem_u32(sB + stage * kBStageBytes));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16(d_tmem, da + 2u * k, db + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&empty[stage]);
          if (++stage == NS) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(&tfull[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> swizzled smem box -> TMA store / reduce (both CTAs) ----
    const int quad = warp & 3;                       // TMEM lane quarter this warp may read
    const int cgrp = (warp - 2) >> 2;                // which 64-column group of the tile
    uint8_t* buf = boxes + (warp - 2) * kOutBoxBytes;
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmD)) : "memory");
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int64_t q = cluster_id; q < pieces; q += n_clusters) {
      const Piece pc = piece_of(q / ks, tiles, tail);
      const int64_t m0 = (pc.tile % m_tiles) * BM + rank * kRowsPerCta, n0 = (pc.tile / m_tiles) * BN + pc.noff;
      if (!mbar_wait(&tfull[acc], acc_phase, g.status)) break;
      tc_fence_after();
      const int row0 = static_cast<int>(m0) + quad * 32;
      const int plane0 = static_cast<int>((q % ks) * g.plane_rows);      // first output row of this piece's range of K
      const int col0 = static_cast<int>(n0) + cgrp * kColsPerEpiWarp;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                             static_cast<uint32_t>(acc * BN + cgrp * kColsPerEpiWarp);
      // (a half piece fills the first 128 accumulator columns: the warps of the other two column groups only arrive)
      if (cgrp * kColsPerEpiWarp < pc.nw && row0 < M_rows && (col0 < g.N || EPI == kEpiArgmax))
        epilogue_columns<EPI>(g, &tmD, buf, lane, taddr, ks > 1 ? plane0 + row0 : row0, col0);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa(smem_u32(&tempty[acc]), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();                  // the staged boxes must be out before shared memory goes away
  }

  // Both CTAs stay until the pair is done: the leader's MMAs read the peer's shared memory and
  // write its tensor memory, and the peer signals barriers that live in the leader.
  tc_fence_before();
  cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace tc
}  // namespace srm
