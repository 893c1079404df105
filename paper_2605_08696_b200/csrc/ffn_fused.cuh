// The feed-forward block of one layer as ONE kernel:  H = gelu(a W1^T + b1);  x += H W2^T + b2.
//
// Same machinery as gemm_tc_kernel (CTA pairs, 256 x 256 tiles, TMA operand ring, tcgen05.mma with two accumulators
// in tensor memory, 16 epilogue warps with bulk-tensor stores / reduce-adds), but the tiles of BOTH projections are
// dealt to the pairs by a plan made on the host (ffn_plan.h) and passed as a launch parameter. Two launches lose a
// ramp and a drain each (the last epilogue of every pair runs beside nothing), and with 64 down tiles for 74 pairs
// ten pairs idle through the whole down projection; here those pairs keep computing up tiles while the others are
// already in their down tile.
//
// What makes that possible: a down tile reads H[row block, :] along its K dimension, column tile after column
// tile, so it needs an up tile only when its k-loop gets there. Every up tile has a counter in global memory; each
// of its 32 epilogue warps (both CTAs) adds one after its bulk stores have completed (release), and the TMA
// producer of a down tile waits for 32 (acquire) before it loads the first k-block of that column tile. The
// counters are zero on entry (the host clears the whole array once per decode step; every layer has its own).
// Results are those of the two launches bit for bit: every tile is computed whole, by one pair, in the same
// k-order, and every element of x gets one add.
//
// The pairs wait for one another, so all of them must be resident at once: the grid is the number of pairs the
// device holds (one CTA per SM), and nothing else of this library shares the SMs while it runs (kernels of one
// stream run in order). Every wait is bounded all the same: a pair that gives up raises kStatusWaitTimeout and
// leaves its loops; the others time out in turn and the kernel ends.
#pragma once

#include "ffn_plan.h"
#include "gemm_tc.cuh"
#include "gemm_tc_splitk.cuh"   // ld_acquire_gpu, fence_async_global, kOrderWaitLimitCycles

namespace srm {
namespace tc {

constexpr int kFfnReadyArrivals = 2 * kEpiWarps;     // epilogue warps of both CTAs of a pair

struct FfnArgs {
  int64_t M;             // rows
  int d, F;              // model width, hidden width
  const float* b1;       // [F]
  const float* b2;       // [d]
  uint32_t* status;
  int32_t* ready;        // [ceil(M / 256)][F / 256] counters, zero on entry
  int w_static;          // W1, W2 are constant data: the first tiles may be fetched ahead of the dependency wait
};

__device__ __forceinline__ void red_release_add(int32_t* p, int32_t v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Waits until the counter has reached `want`. Sleeps between tries: a waiting producer must not take issue slots
// (or power) from the pairs that compute what it waits for.
__device__ __forceinline__ bool ready_wait(const int32_t* p, int32_t want, uint32_t* status) {
  if (ld_acquire_gpu(p) >= want) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      __nanosleep(200);
      if (ld_acquire_gpu(p) >= want) return true;
    }
    if (clock64() - t0 > kOrderWaitLimitCycles) {
      raise_status(status, kStatusWaitTimeout);
      return false;
    }
  }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
ffn_fused_kernel(const __grid_constant__ CUtensorMap tmA,     // a   [M, d] bf16, load boxes of 128 rows
                 const __grid_constant__ CUtensorMap tmW1,    // W1  [F, d]
                 const __grid_constant__ CUtensorMap tmW1h,   // W1, load boxes of 64 rows (half-width pieces)
                 const __grid_constant__ CUtensorMap tmHs,    // H   [M, F] bf16, store boxes of 32 rows
                 const __grid_constant__ CUtensorMap tmH,     // H, load boxes of 128 rows
                 const __grid_constant__ CUtensorMap tmW2,    // W2  [d, F]
                 const __grid_constant__ CUtensorMap tmX,     // x   [M, d] fp32, reduce-add boxes of 32 rows
                 const FfnArgs g, const __grid_constant__ FfnPlan plan) {
  pdl_trigger();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + kStages * kAStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes + kEpiWarps * kOutBoxBytes);
  uint64_t* empty = full + kStages;
  uint64_t* tfull = empty + kStages;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  uint8_t* boxes = smem + kStages * kStageBytes;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
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
  if (threadIdx.x != 0) pdl_wait();

  const int i0 = cluster_id < plan.n_pairs ? plan.off[cluster_id] : 0;
  const int i1 = cluster_id < plan.n_pairs ? plan.off[cluster_id + 1] : 0;
  const int kb_up = g.d / BK, kb_dn = g.F / BK;
  const int Cu = g.F / BN;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmW1)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmH)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmW2)) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // While the predecessor kernel drains: the weight halves of the first stages of the first item.
      int pre = 0;
      if (i0 < i1 && g.w_static) {
        const uint16_t it = plan.item[i0];
        const bool down = ffn_item_down(it), half = ffn_item_half(it);
        const int kbs = down ? kb_dn : kb_up;
        const int w_rows = half ? kHalfN / 2 : kRowsPerCta;               // W rows each CTA of the pair loads
        const int n_row = ffn_item_cb(it) * BN + ffn_item_noff(it) + (int)rank * w_rows;
        pre = kbs < kStages ? kbs : kStages;
        for (int i = 0; i < pre; ++i) {
          const uint32_t full_leader = mapa(smem_u32(&full[i]), 0);
          mbar_expect_tx_cluster(full_leader, kAStageBytes + (uint32_t)w_rows * BK * 2);
          tma_load_2d(sB + i * kBStageBytes, down ? &tmW2 : (half ? &tmW1h : &tmW1), full_leader, i * BK, n_row);
        }
      }
      pdl_wait();
      for (int i = i0; ok && i < i1; ++i) {
        const uint16_t it = plan.item[i];
        const bool down = ffn_item_down(it), half = ffn_item_half(it);
        const int rb = ffn_item_rb(it);
        const int kbs = down ? kb_dn : kb_up;
        const int w_rows = half ? kHalfN / 2 : kRowsPerCta;
        const uint32_t stage_bytes = kAStageBytes + (uint32_t)w_rows * BK * 2;
        const CUtensorMap* mapA = down ? &tmH : &tmA;
        const CUtensorMap* mapB = down ? &tmW2 : (half ? &tmW1h : &tmW1);
        const int m_row = rb * BM + (int)rank * kRowsPerCta;
        const int n_row = ffn_item_cb(it) * BN + ffn_item_noff(it) + (int)rank * w_rows;
        const int32_t* rdy = g.ready + (int64_t)rb * Cu;
        for (int kb = 0; kb < kbs; ++kb) {
          const uint32_t full_leader = mapa(smem_u32(&full[stage]), 0);
          if (pre > 0) {
            --pre;
          } else {
            if (!mbar_wait(&empty[stage], phase ^ 1u, g.status)) { ok = false; break; }
            mbar_expect_tx_cluster(full_leader, stage_bytes);
            tma_load_2d(sB + stage * kBStageBytes, mapB, full_leader, kb * BK, n_row);
          }
          if (down && (kb % kFfnKbPerHTile) == 0) {
            // column tile kb / 4 of H[rb, :] must be complete: all epilogue warps of the pair that computed it
            if (!ready_wait(rdy + kb / kFfnKbPerHTile, kFfnReadyArrivals, g.status)) { ok = false; break; }
            fence_async_global();
          }
          tma_load_2d(sA + stage * kAStageBytes, mapA, full_leader, kb * BK, m_row);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
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
      for (int i = i0; ok && i < i1; ++i) {
        const int kbs = ffn_item_down(plan.item[i]) ? kb_dn : kb_up;
        const uint32_t idesc = ffn_item_half(plan.item[i]) ? instr_desc(kHalfN) : kInstrDesc;
        if (!mbar_wait(&tempty[acc], acc_phase ^ 1u, g.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = 0; kb < kbs; ++kb) {
          if (!mbar_wait(&full[stage], phase, g.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = make_smem_desc(smem_u32(sA + stage * kAStageBytes));
          const uint64_t db = make_smem_desc(smem_u32(sB + stage * kBStageBytes));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16(d_tmem, da + 2u * k, db + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(&tfull[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue (both CTAs) ----------------
    const int quad = warp & 3;
    const int cgrp = (warp - 2) >> 2;
    uint8_t* buf = boxes + (warp - 2) * kOutBoxBytes;
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmHs)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
    }
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int i = i0; i < i1; ++i) {
      const uint16_t it = plan.item[i];
      const bool down = ffn_item_down(it);
      const int rb = ffn_item_rb(it), cb = ffn_item_cb(it);
      if (!mbar_wait(&tfull[acc], acc_phase, g.status)) break;
      tc_fence_after();
      const int row0 = rb * BM + (int)rank * kRowsPerCta + quad * 32;
      const int col0 = cb * BN + ffn_item_noff(it) + cgrp * kColsPerEpiWarp;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                             static_cast<uint32_t>(acc * BN + cgrp * kColsPerEpiWarp);
      // (a half piece fills the first 128 accumulator columns: the warps of the other two column groups only arrive)
      const bool mine = !ffn_item_half(it) || cgrp * kColsPerEpiWarp < kHalfN;
      if (row0 < g.M && mine) {
        if (down) {
          const GemmArgs ga{g.M, g.d, g.F, g.b2, nullptr, g.status, 0};
          epilogue_columns<kEpiBiasResidual>(ga, &tmX, buf, lane, taddr, row0, col0);
        } else {
          const GemmArgs ga{g.M, g.F, g.d, g.b1, nullptr, g.status, 0};
          epilogue_columns<kEpiBiasGelu>(ga, &tmHs, buf, lane, taddr, row0, col0);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_cluster(mapa(smem_u32(&tempty[acc]), 0));
        if (!down && mine) {
          // this warp's part of the H tile is in global memory: count it in (the next accumulator is a tile's
          // main loop away, so the wait for the store costs nothing); the two halves of a tile computed in halves
          // count 16 warps each
          bulk_wait_all();
          fence_async_global();
          red_release_add(g.ready + (int64_t)rb * Cu + cb, 1);
        }
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();
  }

  tc_fence_before();
  cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace tc
}  // namespace srm
