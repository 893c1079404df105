// bf16 projection D[M,N] = A[M,K] * W[N,K]^T on the 5th-generation tensor cores (sm_100a):
// TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) -> shared-memory ring ->
// tcgen05.mma (one issuing thread, cta_group::1, 128x256x16 per instruction) with fp32
// accumulators in tensor memory (two 256-column buffers, so the epilogue of tile i overlaps
// the main loop of tile i+1) -> tcgen05.ld -> fused epilogue -> global memory.
//
// The kernel is persistent: grid = min(tiles, SMs), tiles are taken round-robin.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue
// (warp w reads TMEM lanes 32*(w%4) .. +31, i.e. one accumulator row per thread).
// Every wait is bounded: after ~2^31 clock cycles a waiter raises kStatusWaitTimeout, leaves its
// loop, and the CTA still releases its tensor memory and exits.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "gemm_simt.cuh"   // GemmEpilogue enum

namespace srm {
namespace tc {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kStages = 4;
constexpr int kAStageBytes = BM * BK * 2;        // 16 KiB
constexpr int kBStageBytes = BN * BK * 2;        // 32 KiB
constexpr int kStageBytes = kAStageBytes + kBStageBytes;
constexpr int kBarrierBytes = 256;
constexpr int kSmemBytes = kStages * kStageBytes + kBarrierBytes + 1024;  // +1024: manual alignment
constexpr int kThreads = 192;
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
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false (after raising the status bit) when the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > kWaitLimitCycles) {
      raise_status(status, kStatusWaitTimeout);
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrive once all tcgen05 operations issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
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
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

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
// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = BN, M = BM.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(BN >> 3) << 17) |
                                (uint32_t(BM >> 4) << 24);

struct GemmArgs {
  int64_t M, N, K;
  const float* bias;   // [N] (epilogues 0, 1)
  void* out;           // bf16 [M,N] (epilogue 0) or float [M,N] (epilogues 1, 2)
  uint32_t* status;
};

template <int EPI>
__device__ __forceinline__ void epilogue_store(const GemmArgs& g, int64_t row, int64_t col0, const uint32_t (&r)[32]) {
  if (row >= g.M) return;
  if (EPI == kEpiBiasGelu) {
    bf16* o = reinterpret_cast<bf16*>(g.out) + row * g.N + col0;
#pragma unroll
    for (int j = 0; j < 32; j += 8) {
      if (col0 + j < g.N) {
        const float4 b0 = __ldg(reinterpret_cast<const float4*>(g.bias + col0 + j));
        const float4 b1 = __ldg(reinterpret_cast<const float4*>(g.bias + col0 + j + 4));
        __nv_bfloat162 p0 = __floats2bfloat162_rn(gelu_erf(__uint_as_float(r[j + 0]) + b0.x),
                                                  gelu_erf(__uint_as_float(r[j + 1]) + b0.y));
        __nv_bfloat162 p1 = __floats2bfloat162_rn(gelu_erf(__uint_as_float(r[j + 2]) + b0.z),
                                                  gelu_erf(__uint_as_float(r[j + 3]) + b0.w));
        __nv_bfloat162 p2 = __floats2bfloat162_rn(gelu_erf(__uint_as_float(r[j + 4]) + b1.x),
                                                  gelu_erf(__uint_as_float(r[j + 5]) + b1.y));
        __nv_bfloat162 p3 = __floats2bfloat162_rn(gelu_erf(__uint_as_float(r[j + 6]) + b1.z),
                                                  gelu_erf(__uint_as_float(r[j + 7]) + b1.w));
        uint4 u;
        u.x = *reinterpret_cast<uint32_t*>(&p0); u.y = *reinterpret_cast<uint32_t*>(&p1);
        u.z = *reinterpret_cast<uint32_t*>(&p2); u.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(o + j) = u;
      }
    }
  } else {
    float* o = reinterpret_cast<float*>(g.out) + row * g.N + col0;
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
      if (col0 + j < g.N) {
        float4 v = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                               __uint_as_float(r[j + 3]));
        if (EPI == kEpiBiasResidual) {
          const float4 b = __ldg(reinterpret_cast<const float4*>(g.bias + col0 + j));
          const float4 x = *reinterpret_cast<const float4*>(o + j);
          v = make_float4(x.x + (v.x + b.x), x.y + (v.y + b.y), x.z + (v.z + b.z), x.w + (v.w + b.w));
        }
        *reinterpret_cast<float4*>(o + j) = v;
      }
    }
  }
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + kStages * kAStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* empty = full + kStages;
  uint64_t* tfull = empty + kStages;     // [2] accumulator ready for the epilogue
  uint64_t* tempty = tfull + 2;          // [2] accumulator drained by the epilogue
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 128); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int64_t m_tiles = (g.M + BM - 1) / BM, n_tiles = (g.N + BN - 1) / BN;
  const int64_t tiles = m_tiles * n_tiles;
  const int k_blocks = static_cast<int>(g.K / BK);

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; ok && tile < tiles; tile += gridDim.x) {
        const int m0 = static_cast<int>(tile % m_tiles) * BM, n0 = static_cast<int>(tile / m_tiles) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1u, g.status)) { ok = false; break; }
          mbar_expect_tx(&full[stage], kStageBytes);
          tma_load_2d(sA + stage * kAStageBytes, &tmA, &full[stage], kb * BK, m0);
          tma_load_2d(sB + stage * kBStageBytes, &tmB, &full[stage], kb * BK, n0);
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // another role gave up: let the copies already issued land before the CTA exits
        const int pending = issued < kStages ? issued : kStages;
        for (int i = 0; i < pending; ++i) {
          if (stage == 0) { stage = kStages; phase ^= 1u; }
          --stage;
          (void)mbar_wait(&full[stage], phase, nullptr);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; ok && tile < tiles; tile += gridDim.x) {
        if (!mbar_wait(&tempty[acc], acc_phase ^ 1u, g.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&full[stage], phase, g.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = make_smem_desc(smem_u32(sA + stage * kAStageBytes));
          const uint64_t db = make_smem_desc(smem_u32(sB + stage * kBStageBytes));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16(d_tmem, da + 2u * k, db + 2u * k, kInstrDesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(&empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&tfull[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    const int quad = warp & 3;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
      const int64_t m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
      if (!mbar_wait(&tfull[acc], acc_phase, g.status)) break;
      tc_fence_after();
      const int64_t row = m0 + quad * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(acc * BN);
#pragma unroll 1
      for (int c = 0; c < BN; c += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + c, r);
        tmem_ld_wait();
        if (n0 + c < g.N) epilogue_store<EPI>(g, row, n0 + c, r);
      }
      tc_fence_before();
      mbar_arrive(&tempty[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace tc
}  // namespace srm
