// Temperature + nucleus (top-p) sampling over the vocabulary (Holtzman et al., ICLR 2020; the sampler of
// the paper's GRPO rollouts: Training details, top-p 0.9 at temperature 0.7).
//
// Definition (one row of logits l_v): probabilities softmax(l / T); the nucleus is the shortest prefix of
// the order (logit descending, id ascending) whose probability mass reaches p; the token is drawn from the
// nucleus by inverse CDF over ids in ascending order with u = Philox4x32-10(seed; sample, step).
//
// A nucleus can hold most of the vocabulary (flat distributions), so nothing here sorts the row.
//   * Weights are fixed-point integers q_v = round(2^31 exp((l_v - max) / T)) and every mass is an exact
//     64-bit integer sum: sums do not depend on the order of addition, so neither the nucleus nor the drawn
//     token depends on thread scheduling, and thresholds are compared exactly.
//   * The last nucleus member is located with one histogram pass: mass and count of 2048 buckets evenly
//     spaced in logit value between the smallest logit of non-zero weight and the maximum (shared-memory
//     atomics; with that many buckets neighbouring tokens rarely meet), a block-wide suffix sum over the
//     buckets finds the one in which the cumulative mass from the top crosses p Z, and its few dozen tokens
//     are ranked exactly (ties by id). Only when more tokens share that bucket than the exact stage holds
//     (heavy ties) a four-way search on the bucket's key range follows: each pass sums mass and count of the
//     range's four parts (pivots evenly spaced in logit value while the range is wide, in key space
//     afterwards, which bounds the passes) until at most kToppExact tokens or a single key (all ties) remain.
//   * The draw scans the row in id order: every thread owns a contiguous chunk, two block-wide prefix sums
//     (ties before the chunk, nucleus mass before the chunk) locate the thread that holds the token.
// One block per row; the row's keys are staged in shared memory when they fit (V <= kToppSmemFloats), else
// the row is re-read from global memory (L2) on every pass.
#pragma once

#include "common.cuh"
#include "select.cuh"

namespace srm {

constexpr int kToppThreads = 1024;
constexpr int kToppWarps = kToppThreads / 32;
constexpr int kToppCap = 1024;                   // capacity of the exact last stage (one token per thread)
constexpr int kToppExact = 256;                  // the search stops when the part that holds the edge has this few tokens
                                                 // (ranking n candidates costs n^2 comparisons)
constexpr int kToppMaxPasses = 28;               // 6 passes with value pivots, then 4-way search on at most 2^32 keys
constexpr int kToppSmemFloats = 40 * 1024;       // rows up to 160 KB are staged in shared memory
constexpr int kToppBuckets = 2048;               // histogram buckets (two per thread in the suffix sum)
constexpr float kToppFixedOne = 2147483648.0f;   // 2^31: weight of the most probable token (weights fit 32 bits)

struct ToppScratch {
  unsigned long long red[kToppWarps][8];         // block reductions: 4 masses + 4 counts
  unsigned long long scan[kToppWarps];           // block prefix sums
  unsigned long long scan_total;
  unsigned long long bcast[8];
  uint32_t ckey[kToppCap], skey[kToppCap];
  int32_t cid[kToppCap], sid[kToppCap];
  unsigned long long cq[kToppCap], sq[kToppCap];
  int n_cand, pos, first, bstar, n_ties;
  unsigned int kmin, kmax;
  float fmax_w[kToppWarps], fmin_w[kToppWarps];
};

// round(2^31 exp((l - m) / T)) = round(2^(31 + (l - m) s)), s = log2(e) / T: one fused multiply-add, the
// hardware exp2 (relative error 2^-22, well inside the tolerance of the comparison with the oracle), one
// conversion. Arguments below -1 give less than one half and round to zero; NaN converts to zero.
__device__ __forceinline__ unsigned long long topp_weight(float l, float m, float s) {
  const float x = fmaf(l - m, s, 31.0f);
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x));
  return (unsigned long long)__float2uint_rn(e);
}
struct ToppHist {
  unsigned long long mass[kToppBuckets];
  unsigned int cnt[kToppBuckets];
};

// NaN sorts below everything
__device__ __forceinline__ uint32_t topp_key(float l) { return (l == l) ? order_key(l) : 0u; }

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// exclusive prefix sum of one value per thread over the block; `total` receives the block sum
__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long v, ToppScratch* sc,
                                                                   unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();                               // previous users of sc->scan are done
  if (lane == 31) sc->scan[warp] = incl;
  __syncthreads();
  if (warp == 0) {                               // exclusive scan of the warp totals (lane = warp index)
    const unsigned long long t = lane < kToppWarps ? sc->scan[lane] : 0ull;
    unsigned long long ti = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long u = __shfl_up_sync(0xffffffffu, ti, o);
      if (lane >= o) ti += u;
    }
    if (lane < kToppWarps) sc->scan[lane] = ti - t;
    if (lane == 31) sc->scan_total = ti;
  }
  __syncthreads();
  *total = sc->scan_total;
  return sc->scan[warp] + incl - v;
}

template <bool ROW_IN_SMEM>
__global__ void __launch_bounds__(kToppThreads)
select_topp_kernel(const float* __restrict__ logits, int64_t R, int V, float top_p, float inv_temp, uint64_t seed,
                   uint64_t sample_base, int step, SelectOut out, uint32_t* status) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ __align__(16) uint8_t topp_smem[];
  ToppScratch* sc = reinterpret_cast<ToppScratch*>(topp_smem);
  ToppHist* hist = reinterpret_cast<ToppHist*>(topp_smem + ((sizeof(ToppScratch) + 15) & ~size_t(15)));
  uint32_t* skeys = reinterpret_cast<uint32_t*>(topp_smem + ((sizeof(ToppScratch) + 15) & ~size_t(15)) + sizeof(ToppHist));
  const int64_t row = blockIdx.x;
  if (row >= R) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* grow = logits + (row / out.row_div) * (int64_t)V;

  // ---- pass 0: stage the row, maximum (NaN ignored, flagged) ----
  float mx = -INFINITY, mn = INFINITY;
  bool bad = false;
  for (int i = tid; i < V; i += kToppThreads) {
    const float l = grow[i];
    if (ROW_IN_SMEM) skeys[i] = topp_key(l);
    bad |= !(fabsf(l) <= 3.0e38f);               // NaN or infinity
    if (l > mx) mx = l;
    if (l < mn) mn = l;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  }
  if (lane == 0) { sc->fmax_w[warp] = mx; sc->fmin_w[warp] = mn; }
  if (bad) raise_status(status, kStatusNonFinite);
  __syncthreads();
  if (warp == 0) {
    mx = lane < kToppWarps ? sc->fmax_w[lane] : -INFINITY;
    mn = lane < kToppWarps ? sc->fmin_w[lane] : INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    }
    if (lane == 0) { sc->fmax_w[0] = mx; sc->fmin_w[0] = mn; }
  }
  __syncthreads();
  mx = sc->fmax_w[0]; mn = sc->fmin_w[0];
  auto key_at = [&](int i) -> uint32_t { return ROW_IN_SMEM ? skeys[i] : topp_key(grow[i]); };
  if (!(mx > -INFINITY) || !(mx < INFINITY)) {   // no finite maximum: nothing to sample from
    if (tid == 0) write_token(out, row, 0);
    return;
  }

  const float s = inv_temp * 1.4426950408889634f;
  // search range [lo, hi) in key space; `above` = mass of the keys >= hi
  // (tokens more than 33 / s below the maximum have weight zero; nothing lies below the row's minimum)
  const float lo_v = fmaxf(mx - 33.0f / s, mn);
  uint64_t lo = topp_key(lo_v), hi = (uint64_t)topp_key(mx) + 1;
  unsigned long long above = 0, target = 0, in_mass = 0;
  long long in_cnt = 0;

  // ---- histogram over logit value: the bucket in which the cumulative mass from the top reaches p Z ----
  const float b_scale = mx > lo_v ? (float)kToppBuckets / (mx - lo_v) : 0.f;
  auto bucket_of = [&](float l) -> int {         // monotone in l; -1 for weight-zero tokens and NaN
    if (!(l >= lo_v)) return -1;
    const int b = (int)((l - lo_v) * b_scale);
    return b < kToppBuckets ? b : kToppBuckets - 1;
  };
  for (int i = tid; i < kToppBuckets; i += kToppThreads) { hist->mass[i] = 0ull; hist->cnt[i] = 0u; }
  if (tid == 0) { sc->bstar = kToppBuckets - 1; sc->bcast[1] = 0ull; }      // (always overwritten: Z >= the maximum's weight)
  __syncthreads();
  for (int i = tid; i < V; i += kToppThreads) {
    const float l = key_value(key_at(i));
    const int b = bucket_of(l);
    if (b >= 0) {
      atomicAdd(&hist->mass[b], topp_weight(l, mx, s));
      atomicAdd(&hist->cnt[b], 1u);
    }
  }
  __syncthreads();
  {
    // thread t owns buckets B-1-2t (upper) and B-2-2t: an exclusive scan over threads is a suffix sum over buckets
    const int bu = kToppBuckets - 1 - 2 * tid, bl = bu - 1;
    const unsigned long long mu = bu >= 0 ? hist->mass[bu] : 0ull, ml = bl >= 0 ? hist->mass[bl] : 0ull;
    unsigned long long Z;
    const unsigned long long before = block_exclusive_scan(mu + ml, sc, &Z);
    // Z: every token of non-zero weight; the mass the nucleus must reach
    const double t = ceil((double)top_p * (double)Z);
    target = t < 1.0 ? 1ull : (t > (double)Z ? Z : (unsigned long long)t);
    if (before < target && target <= before + mu) { sc->bstar = bu; sc->bcast[1] = before; }
    else if (before + mu < target && target <= before + mu + ml) { sc->bstar = bl; sc->bcast[1] = before + mu; }
    __syncthreads();
  }
  const int bstar = sc->bstar;
  above = sc->bcast[1];
  in_cnt = (long long)hist->cnt[bstar];
  in_mass = hist->mass[bstar];
  bool by_keys = false;                        // candidates are selected by key range (after the search) or by bucket
  if (in_cnt > kToppCap) {
    // heavy ties: more tokens in the edge bucket than the exact stage holds. Its key range (bucket_of is
    // monotone, so every key between two of its keys belongs to it), then the four-way search on that range.
    if (tid == 0) { sc->kmin = 0xffffffffu; sc->kmax = 0u; }
    __syncthreads();
    unsigned int kmn = 0xffffffffu, kmx = 0u;
    for (int i = tid; i < V; i += kToppThreads) {
      const uint32_t k = key_at(i);
      if (bucket_of(key_value(k)) == bstar) { kmn = k < kmn ? k : kmn; kmx = k > kmx ? k : kmx; }
    }
    kmn = __reduce_min_sync(0xffffffffu, kmn); kmx = __reduce_max_sync(0xffffffffu, kmx);
    if (lane == 0) { atomicMin(&sc->kmin, kmn); atomicMax(&sc->kmax, kmx); }
    __syncthreads();
    lo = sc->kmin; hi = (uint64_t)sc->kmax + 1;
    by_keys = true;
  }
  for (int pass = 0; by_keys && hi - lo > 1 && pass < kToppMaxPasses; ++pass) {
    // three pivots lo < p1 <= p2 <= p3 < hi (as keys)
    uint32_t pv[3];
    const uint64_t width = hi - lo;
    bool by_value = pass < 6 && width > (1u << 12);
    if (by_value) {
      const float vlo = key_value((uint32_t)lo), vhi = key_value((uint32_t)(hi - 1));
      const float st = (vhi - vlo) * 0.25f;
#pragma unroll
      for (int j = 0; j < 3; ++j) pv[j] = topp_key(vlo + st * (float)(j + 1));
      by_value = (pv[0] > lo) && (pv[0] <= pv[1]) && (pv[1] <= pv[2]) && (pv[2] < hi - 1) && (vhi - vlo < INFINITY);
    }
    if (!by_value) {
      const uint64_t w4 = (width + 3) / 4;
#pragma unroll
      for (int j = 0; j < 3; ++j) {
        const uint64_t pj = lo + w4 * (uint64_t)(j + 1);
        pv[j] = (uint32_t)(pj < hi ? pj : hi - 1);
      }
    }
    const uint32_t p1 = pv[0], p2 = pv[1], p3 = pv[2];
    unsigned long long m0 = 0, m1 = 0, m2 = 0, m3 = 0;
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
    const uint32_t lo32 = (uint32_t)lo, hi32 = (uint32_t)(hi - 1);           // inclusive upper end
    for (int i = tid; i < V; i += kToppThreads) {
      const uint32_t k = key_at(i);
      if (k >= lo32 && k <= hi32) {
        const unsigned long long q = topp_weight(key_value(k), mx, s);
        const int b = (k >= p1) + (k >= p2) + (k >= p3);
        m0 += (b == 0) ? q : 0ull; m1 += (b == 1) ? q : 0ull; m2 += (b == 2) ? q : 0ull; m3 += (b == 3) ? q : 0ull;
        c0 += (b == 0); c1 += (b == 1); c2 += (b == 2); c3 += (b == 3);
      }
    }
    m0 = warp_sum_u64(m0); m1 = warp_sum_u64(m1); m2 = warp_sum_u64(m2); m3 = warp_sum_u64(m3);
    c0 = __reduce_add_sync(0xffffffffu, c0); c1 = __reduce_add_sync(0xffffffffu, c1);
    c2 = __reduce_add_sync(0xffffffffu, c2); c3 = __reduce_add_sync(0xffffffffu, c3);
    __syncthreads();
    if (lane == 0) {
      sc->red[warp][0] = m0; sc->red[warp][1] = m1; sc->red[warp][2] = m2; sc->red[warp][3] = m3;
      sc->red[warp][4] = c0; sc->red[warp][5] = c1; sc->red[warp][6] = c2; sc->red[warp][7] = c3;
    }
    __syncthreads();
    if (warp == 0) {                             // one warp folds the per-warp partials (lane = warp index)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const unsigned long long t = warp_sum_u64(lane < kToppWarps ? sc->red[lane][j] : 0ull);
        if (lane == 0) sc->bcast[j] = t;
      }
    }
    __syncthreads();
    unsigned long long mass[4], cnt[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { mass[j] = sc->bcast[j]; cnt[j] = sc->bcast[4 + j]; }
    // from the top: the part in which the cumulative mass reaches the target
    int chosen = 0;
    unsigned long long acc = above;
#pragma unroll
    for (int b = 3; b >= 0; --b) {
      if (acc + mass[b] >= target) { chosen = b; break; }
      acc += mass[b];
    }
    above = acc;
    const uint64_t nlo = chosen == 0 ? lo : pv[chosen - 1], nhi = chosen == 3 ? hi : pv[chosen];
    lo = nlo; hi = nhi;
    in_mass = mass[chosen];
    in_cnt = (long long)cnt[chosen];
    if (in_cnt <= kToppExact || hi - lo <= 1) break;
  }

  // ---- the last nucleus member: its key, how many tokens of that key are in, the nucleus mass ----
  uint32_t kstar;
  long long n_ties_in, n_ties_all;             // tokens of the edge key that are in the nucleus / that exist
  unsigned long long nucleus_mass;
  if (in_cnt <= kToppCap) {
    if (tid == 0) { sc->n_cand = 0; sc->pos = kToppCap; sc->first = kToppCap; sc->n_ties = 0; }
    __syncthreads();
    for (int i = tid; i < V; i += kToppThreads) {
      const uint32_t k = key_at(i);
      if (by_keys ? (k >= lo && k < hi) : (bucket_of(key_value(k)) == bstar)) {
        const int slot = atomicAdd(&sc->n_cand, 1);
        if (slot < kToppCap) { sc->ckey[slot] = k; sc->cid[slot] = i; sc->cq[slot] = topp_weight(key_value(k), mx, s); }
      }
    }
    __syncthreads();
    const int n = sc->n_cand < kToppCap ? sc->n_cand : kToppCap;
    if (tid < n) {                               // rank by (key descending, id ascending)
      const uint32_t kt = sc->ckey[tid];
      const int it = sc->cid[tid];
      int rank = 0;
      for (int j = 0; j < n; ++j) rank += (sc->ckey[j] > kt) || (sc->ckey[j] == kt && sc->cid[j] < it);
      sc->skey[rank] = kt; sc->sid[rank] = it; sc->sq[rank] = sc->cq[tid];
    }
    __syncthreads();
    unsigned long long tot;
    const unsigned long long mine = tid < n ? sc->sq[tid] : 0ull;
    const unsigned long long before = block_exclusive_scan(mine, sc, &tot);
    if (tid < n && above + before + mine >= target) atomicMin(&sc->pos, tid);
    __syncthreads();
    const int pos = sc->pos < n ? sc->pos : n - 1;     // (n >= 1: the chosen part holds the boundary token)
    kstar = sc->skey[pos];
    if (tid <= pos && sc->skey[tid] == kstar) atomicMin(&sc->first, tid);
    if (tid < n && sc->skey[tid] == kstar) atomicAdd(&sc->n_ties, 1);
    if (tid == pos) sc->bcast[0] = above + before + mine;
    __syncthreads();
    n_ties_in = pos - sc->first + 1;
    n_ties_all = sc->n_ties;
    nucleus_mass = sc->bcast[0];
  } else {
    // a single key with more than kToppCap tokens: all ties, taken in id order
    kstar = (uint32_t)lo;
    const unsigned long long qt = in_mass / (unsigned long long)in_cnt;       // they all carry the same weight
    long long c = qt > 0 ? (long long)((target - above + qt - 1) / qt) : in_cnt;
    n_ties_in = c < 1 ? 1 : (c > in_cnt ? in_cnt : c);
    n_ties_all = in_cnt;
    nucleus_mass = above + (unsigned long long)n_ties_in * qt;
  }

  // ---- the draw: first id whose cumulative nucleus mass exceeds floor(u * nucleus mass) ----
  const uint64_t sidx = sample_base + (uint64_t)row;
  const uint32_t r = philox4x32_10_word0((uint32_t)sidx, (uint32_t)(out.ctr != nullptr ? out.ctr[kCtrStep] : step), 0u, 0u,
                                         (uint32_t)seed, (uint32_t)(seed >> 32));
  const double u = (double)(r >> 8) * (1.0 / 16777216.0);
  const unsigned long long thr = (unsigned long long)(u * (double)nucleus_mass);
  const int chunk = ((V + kToppThreads - 1) / kToppThreads) | 1;             // odd: conflict-free in shared memory
  const int i0 = tid * chunk < V ? tid * chunk : V, i1 = i0 + chunk < V ? i0 + chunk : V;
  // Membership: key above the edge key, or the edge key itself and among its first n_ties_in ids. When all
  // tokens of the edge key are in (the usual case) the count of ties before a chunk is not needed.
  const bool all_ties = n_ties_in >= n_ties_all;
  unsigned long long tot, ties_before = 0;
  if (!all_ties) {
    unsigned long long my_ties = 0;
    for (int i = i0; i < i1; ++i) my_ties += key_at(i) == kstar;
    ties_before = block_exclusive_scan(my_ties, sc, &tot);
  }
  unsigned long long my_mass = 0;
  {
    long long t = (long long)ties_before;
    for (int i = i0; i < i1; ++i) {
      const uint32_t k = key_at(i);
      const bool in = k > kstar || (k == kstar && (all_ties || t++ < n_ties_in));
      if (in) my_mass += topp_weight(key_value(k), mx, s);
    }
  }
  if (tid == 0) sc->pos = -1;
  const unsigned long long mass_before = block_exclusive_scan(my_mass, sc, &tot);      // (barriers inside)
  if (thr >= mass_before && thr < mass_before + my_mass) {
    unsigned long long c = mass_before;
    long long t = (long long)ties_before;
    int pick = -1;
    for (int i = i0; i < i1; ++i) {
      const uint32_t k = key_at(i);
      const bool in = k > kstar || (k == kstar && (all_ties || t++ < n_ties_in));
      if (in) {
        c += topp_weight(key_value(k), mx, s);
        if (c > thr) { pick = i; break; }
      }
    }
    if (pick >= 0) {
      write_token(out, row, pick);
      sc->pos = pick;
    }
  }
  __syncthreads();
  if (tid == 0 && sc->pos < 0) {                  // cannot happen while the sums above are consistent
    raise_status(status, kStatusNonFinite);
    write_token(out, row, 0);
  }
}

}  // namespace srm
