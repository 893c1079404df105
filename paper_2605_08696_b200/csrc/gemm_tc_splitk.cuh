// Down projection x += H W2^T + b2 with the K dimension shared out between CTA pairs.
//
// gemm_tc_kernel gives every CTA pair whole 256 x 256 tiles. With 74 pairs, the 64 tiles of a 4096-row
// batch leave 10 pairs idle for the whole kernel, and 128 or 192 tiles take 2 or 3 rounds of which the
// last is partly empty: an eighth of the tensor time in each case. This epilogue ADDS into the residual
// stream, so a tile's product can be formed in pieces: here the (tile, k-block) sequence is cut into one
// contiguous range per pair, all of (nearly) equal length, and a pair adds the partial product of every
// piece of its range into x with the bulk reduce-add of the unsplit kernel.
//
// Reproducible results need the pieces of one tile added in a fixed order. The ranges are laid out so that
// a tile is never cut more than once, i.e. has at most two pieces: its upper k-range is the FIRST piece of
// one pair's range (finished early in the kernel), its lower k-range the LAST piece of the previous pair's
// range (finished at the end). The lower piece waits, per epilogue warp, for a word in global memory that
// the upper piece's warp releases once its reduce-adds have completed; by then that happened long ago, so
// the order costs nothing. (With more pairs than tiles, equal ranges would cut some tiles twice and put a
// pair's whole range in the middle of a tile, finishing together with its neighbour's last piece: there
// the pairs are grouped, t tiles to t + 1 pairs, which cuts every tile exactly once, and the group's last
// pair, whose single piece is the upper part of the group's last tile, gets a slightly shorter range so
// that it is done before the piece that must follow it.)
// The words are zero whenever no launch is in flight (the lower piece puts its word back to zero).
// Every wait is bounded: on a time-out the waiter raises kStatusWaitTimeout and goes on without the add.
#pragma once

#include "gemm_tc.cuh"

namespace srm {
namespace tc {

constexpr int kSplitSnapKb = 3;        // a cut this close to a tile boundary moves onto it
constexpr int kSplitLead = 12;         // k-blocks by which a group's last pair finishes early
constexpr long long kOrderWaitLimitCycles = 1ll << 30;

struct SplitPlan {
  int tiles, kb;            // output tiles, k-blocks per tile
  int pairs;                // CTA pairs that take part
  int groups;               // 0: one run of equal ranges over all tiles; else tiles < pairs, grouped
  int t_small, n_big;       // grouped: groups 0 .. n_big-1 hold t_small + 1 tiles, the rest t_small
};

// Whether the split kernel applies, and with how many of the `resident` pairs.
__host__ __device__ inline bool split_plan(int64_t tiles, int kb, int resident, SplitPlan* P) {
  P->tiles = (int)tiles; P->kb = kb; P->pairs = resident; P->groups = 0; P->t_small = 0; P->n_big = 0;
  if (tiles < 1 || kb < 8 || resident < 2) return false;
  if (tiles >= resident) {
    // ranges of at least one tile: never two cuts in one tile. Worth it only if the rounding loss is real.
    const int64_t rounds = (tiles + resident - 1) / resident;
    return rounds * resident - tiles >= resident / 16 && tiles * (int64_t)kb < (1ll << 30);
  }
  const int extra = resident - (int)tiles;               // every group is t tiles for t + 1 pairs
  if (extra > tiles) return false;                       // more than two pairs per tile: not handled
  if (extra < resident / 16) return false;
  P->groups = extra;
  P->t_small = (int)tiles / extra;
  P->n_big = (int)tiles % extra;
  // every cut must stay inside its tile after the last pair's range was shortened, and that range must stay long
  // enough to be worth a pair (checked for the larger groups, which have the shorter ranges per tile)
  const int t = P->t_small + (P->n_big > 0 ? 1 : 0);
  return P->t_small >= 1 && kb / (t + 1) > kSplitLead / P->t_small + 1 && P->t_small * kb / (P->t_small + 1) >= kSplitLead + 8;
}

// k-blocks the longest range is shorter than whole tiles per pair would be. Measured (74 pairs): every extra
// piece costs an epilogue that slows the MMAs running beside it and 256 KB more of reduce-adds in L2; with 9
// or 17 k-blocks saved (64 or 128 tiles of 64 k-blocks) the split kernel is 3 to 4 us slower than the unsplit
// one, with 39 saved (192 tiles of 96) it is 36 us faster. The decode step splits from kSplitWorthKb up.
constexpr int kSplitWorthKb = 32;
__host__ __device__ inline int64_t split_saved_kb(const SplitPlan& P) {
  const int64_t rounds = (P.tiles + P.pairs - 1) / P.pairs;
  const int64_t longest = P.groups == 0 ? ((int64_t)P.tiles * P.kb + P.pairs - 1) / P.pairs + kSplitSnapKb
                                        : (int64_t)P.kb * (P.t_small + 1) / (P.t_small + 2) + kSplitLead;
  return rounds * P.kb - longest;
}

// Range [u0, u1) of pair `c` in units of k-blocks of the (tile-major) sequence.
__host__ __device__ inline void split_range(const SplitPlan& P, int c, int64_t* u0, int64_t* u1) {
  if (P.groups == 0) {
    const int64_t Q = (int64_t)P.tiles * P.kb;
    int64_t b[2];
    for (int i = 0; i < 2; ++i) {
      int64_t v = (int64_t)(c + i) * Q / P.pairs;
      const int rem = (int)(v % P.kb);
      if (rem <= kSplitSnapKb) v -= rem;
      else if (rem >= P.kb - kSplitSnapKb) v += P.kb - rem;
      b[i] = v;
    }
    *u0 = b[0]; *u1 = b[1];
    return;
  }
  // group g: tiles [tile0, tile0 + t), pairs [pair0, pair0 + t + 1)
  const int big_pairs = P.n_big * (P.t_small + 2);
  int g, t, pair0, tile0;
  if (c < big_pairs) {
    t = P.t_small + 1; g = c / (t + 1); pair0 = g * (t + 1); tile0 = g * t;
  } else {
    t = P.t_small;
    const int cc = c - big_pairs;
    g = cc / (t + 1); pair0 = big_pairs + g * (t + 1); tile0 = P.n_big * (P.t_small + 1) + g * t;
  }
  const int k = c - pair0;                               // 0 .. t
  const int64_t total = (int64_t)t * P.kb;
  const int64_t short_last = total / (t + 1) - kSplitLead;            // the last pair's range
  // cuts 1 .. t spread evenly over what is left for the first t pairs
  auto cut = [&](int i) -> int64_t { return i <= 0 ? 0 : (i > t ? total : (int64_t)i * (total - short_last) / t); };
  *u0 = (int64_t)tile0 * P.kb + cut(k);
  *u1 = (int64_t)tile0 * P.kb + cut(k + 1);
}

struct SplitPiece { int tile, kb0, kb1; };

struct SplitCursor {
  int64_t u, u_end;
  __host__ __device__ void init(const SplitPlan& P, int c) { split_range(P, c, &u, &u_end); }
  __host__ __device__ bool next(const SplitPlan& P, SplitPiece* p) {
    if (u >= u_end) return false;
    p->tile = (int)(u / P.kb);
    p->kb0 = (int)(u % P.kb);
    const int64_t left = u_end - u;
    p->kb1 = left < P.kb - p->kb0 ? p->kb0 + (int)left : P.kb;
    u += p->kb1 - p->kb0;
    return true;
  }
};

__host__ __device__ inline size_t split_order_words(int64_t tiles) { return (size_t)tiles * 2 * kEpiWarps; }

struct SplitArgs {
  int64_t M, N, K;
  const float* bias;     // [N] or nullptr
  uint32_t* status;
  int32_t* order;        // [tiles][2][kEpiWarps]: k-blocks of the tile already added, counted from the top
  int w_static;
};

__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t* p) {
  int32_t v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(int32_t* p, int32_t v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// orders accesses made through the generic proxy (the word) and through the async proxy (bulk reduce-add)
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

__device__ __forceinline__ bool order_wait(const int32_t* p, int32_t want, uint32_t* status) {
  if (ld_acquire_gpu(p) == want) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (ld_acquire_gpu(p) == want) return true;
    if (clock64() - t0 > kOrderWaitLimitCycles) {
      raise_status(status, kStatusWaitTimeout);
      return false;
    }
  }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc_splitk_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmD, const SplitArgs g, const SplitPlan P) {
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

  const int m_tiles = (int)((g.M + BM - 1) / BM);       // tile index = n * m_tiles + m, as in gemm_tc_kernel
  SplitCursor cur;
  cur.init(P, cluster_id);
  SplitPiece pc;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      bool have = cur.next(P, &pc);
      int pre = 0;                           // stages of the first piece opened (W in flight) ahead of the dependency wait
      if (have && g.w_static) {
        pre = pc.kb1 - pc.kb0 < kStages ? pc.kb1 - pc.kb0 : kStages;
        const int n_row = (pc.tile / m_tiles) * BN + (int)rank * kRowsPerCta;
        for (int i = 0; i < pre; ++i) {
          const uint32_t full_leader = mapa(smem_u32(&full[i]), 0);
          mbar_expect_tx_cluster(full_leader, kStageBytes);
          tma_load_2d(sB + i * kBStageBytes, &tmB, full_leader, (pc.kb0 + i) * BK, n_row);
        }
      }
      pdl_wait();
      while (have && ok) {
        const int m_row = (pc.tile % m_tiles) * BM + (int)rank * kRowsPerCta;
        const int n_row = (pc.tile / m_tiles) * BN + (int)rank * kRowsPerCta;
        for (int kb = pc.kb0; kb < pc.kb1; ++kb) {
          const uint32_t full_leader = mapa(smem_u32(&full[stage]), 0);
          if (pre > 0) {
            --pre;
          } else {
            if (!mbar_wait(&empty[stage], phase ^ 1u, g.status)) { ok = false; break; }
            mbar_expect_tx_cluster(full_leader, kStageBytes);
            tma_load_2d(sB + stage * kBStageBytes, &tmB, full_leader, kb * BK, n_row);
          }
          tma_load_2d(sA + stage * kAStageBytes, &tmA, full_leader, kb * BK, m_row);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) have = cur.next(P, &pc);
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
      while (ok && cur.next(P, &pc)) {
        if (!mbar_wait(&tempty[acc], acc_phase ^ 1u, g.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = pc.kb0; kb < pc.kb1; ++kb) {
          if (!mbar_wait(&full[stage], phase, g.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = make_smem_desc(smem_u32(sA + stage * kAStageBytes));
          const uint64_t db = make_smem_desc(smem_u32(sB + stage * kBStageBytes));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16(d_tmem, da + 2u * k, db + 2u * k, kInstrDesc, (kb != pc.kb0 || k != 0) ? 1u : 0u);
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
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmD)) : "memory");
    int acc = 0;
    uint32_t acc_phase = 0;
    // the word this warp still has to release once the reduce-adds of its previous piece have completed
    int32_t* pend_ptr = nullptr;
    int32_t pend_val = 0;
    auto publish = [&]() {
      if (pend_ptr != nullptr && lane == 0) {
        bulk_wait_all();
        fence_async_global();
        st_release_gpu(pend_ptr, pend_val);
      }
      pend_ptr = nullptr;
      __syncwarp();
    };
    while (cur.next(P, &pc)) {
      publish();
      if (!mbar_wait(&tfull[acc], acc_phase, g.status)) break;
      tc_fence_after();
      const int row0 = (pc.tile % m_tiles) * BM + (int)rank * kRowsPerCta + quad * 32;
      const int col0 = (pc.tile / m_tiles) * BN + cgrp * kColsPerEpiWarp;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                             static_cast<uint32_t>(acc * BN + cgrp * kColsPerEpiWarp);
      if (row0 < g.M && col0 < g.N) {
        const bool whole = pc.kb0 == 0 && pc.kb1 == P.kb;
        int32_t* word = g.order + ((int64_t)pc.tile * 2 + rank) * kEpiWarps + (warp - 2);
        bool ok = true;
        if (!whole) {
          // everything above this k-range must have been added already
          if (lane == 0) {
            ok = order_wait(word, P.kb - pc.kb1, g.status);
            fence_async_global();
          }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (ok) {
          const GemmArgs ga{g.M, g.N, g.K, pc.kb0 == 0 ? g.bias : nullptr, nullptr, g.status, 0};
          epilogue_columns<kEpiBiasResidual>(ga, &tmD, buf, lane, taddr, row0, col0);
          if (!whole) {
            pend_ptr = word;
            pend_val = pc.kb0 == 0 ? 0 : P.kb - pc.kb0;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa(smem_u32(&tempty[acc]), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    publish();
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
