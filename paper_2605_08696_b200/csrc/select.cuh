// Token selection over the vocabulary: greedy argmax (lowest id among ties) and
// temperature / top-k sampling keyed by Philox4x32-10(seed; sample, step).
// One 256-thread block per sample row; warp-shuffle reductions; the row is streamed with
// 128-bit loads (and staged once in shared memory for the multi-pass top-k selection).
#pragma once

#include "common.cuh"

namespace srm {

constexpr int kSelThreads = 256;
constexpr int kTopKMax = 256;

struct SelectOut {
  int32_t* last_tok;    // [R] always written (state's "previous selection")
  int32_t* tok_out;     // [R] or nullptr
  int32_t* store;       // token store base or nullptr: store[row * store_stride + store_col]
  int64_t store_stride;
  int64_t store_col;
  int64_t row_div;      // output row r reads logits row r / row_div (replicas of one prompt share a row); >= 1
  const int32_t* ctr;   // device-side step counters (store column, Philox step), or nullptr: host values apply
  int32_t* pos;         // [R] per-row positions, advanced by one with every selection, or nullptr
  // Compacted launch (the rows that the fused top-k path hands back): block i serves output row row_map[i] and
  // reads logits row i; only the first *n_rows blocks have work. nullptr: block i serves row i.
  const int32_t* row_map;
  const uint32_t* n_rows;
  float* thr_out;       // [R] or nullptr: top-k only, the candidate threshold to use for this row's next selection
};

// Output row and logits row of block `i`; false when the block has nothing to do.
__device__ __forceinline__ bool select_rows(const SelectOut& o, int64_t i, int64_t R, int64_t* row, int64_t* lrow) {
  if (o.row_map != nullptr) {
    if (i >= (int64_t)*o.n_rows || i >= R) return false;
    *row = o.row_map[i];
    *lrow = i;
    return true;
  }
  if (i >= R) return false;
  *row = i;
  *lrow = i / o.row_div;
  return true;
}

__device__ __forceinline__ void write_token(const SelectOut& o, int64_t row, int tok) {
  o.last_tok[row] = tok;
  if (o.tok_out != nullptr) o.tok_out[row] = tok;
  if (o.store != nullptr) o.store[row * o.store_stride + (o.ctr != nullptr ? (int64_t)o.ctr[kCtrCol] : o.store_col)] = tok;
  if (o.pos != nullptr) o.pos[row] += 1;
}

// ---- greedy -------------------------------------------------------------------------------
__device__ __forceinline__ void argmax_take(float v, int i, float& bv, int& bi) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

__global__ void __launch_bounds__(kSelThreads)
select_greedy_kernel(const float* __restrict__ logits, int64_t R, int V, SelectOut out, uint32_t* status) {
  pdl_trigger();
  pdl_wait();
  const int64_t row = blockIdx.x;
  if (row >= R) return;
  const float* lr = logits + (row / out.row_div) * (int64_t)V;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  bool bad = false;
  for (int i = threadIdx.x * 4; i < V; i += kSelThreads * 4) {
    const float4 v = *reinterpret_cast<const float4*>(lr + i);
    bad |= !(v.x == v.x) | !(v.y == v.y) | !(v.z == v.z) | !(v.w == v.w);
    argmax_take(v.x, i, bv, bi); argmax_take(v.y, i + 1, bv, bi);
    argmax_take(v.z, i + 2, bv, bi); argmax_take(v.w, i + 3, bv, bi);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    argmax_take(ov, oi, bv, bi);
  }
  __shared__ float sv[kSelThreads / 32];
  __shared__ int si[kSelThreads / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
  if (bad) raise_status(status, kStatusNonFinite);
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kSelThreads / 32; ++w) argmax_take(sv[w], si[w], bv, bi);
    if (bi < 0 || bi >= V) bi = 0;       // all-NaN row
    write_token(out, row, bi);
  }
}

// Second stage of the selection fused into the LM head: reduces the per-slice partial results
// part[slot][row] = (bits of the slice maximum, its column) over the slots of each row with the same rule
// (largest value, lowest column among equals). 32 rows x 32 slot lanes per block (with 8 lanes the 128 blocks of a
// 4096-row batch left the kernel latency-bound at 13 us); every load instruction
// of a warp covers 32 consecutive rows (256 contiguous bytes).
constexpr int kArgmaxRows = 32, kArgmaxLanes = 32;
__global__ void __launch_bounds__(kArgmaxRows * kArgmaxLanes)
argmax_reduce_kernel(const uint2* __restrict__ part, int64_t R, int64_t slots, int V, SelectOut out) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sv[kArgmaxLanes][kArgmaxRows];
  __shared__ int si[kArgmaxLanes][kArgmaxRows];
  const int rr = threadIdx.x & 31, sl = threadIdx.x >> 5;
  const int64_t row = (int64_t)blockIdx.x * kArgmaxRows + rr;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  if (row < R) {
    // eight independent loads in flight per thread; slots are visited in ascending order, so the
    // lowest column among equal maxima is kept
    int64_t s = sl;
    for (; s + 7 * kArgmaxLanes < slots; s += 8 * kArgmaxLanes) {
      uint2 q[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) q[u] = __ldg(part + (s + u * kArgmaxLanes) * R + row);
#pragma unroll
      for (int u = 0; u < 8; ++u) argmax_take(__uint_as_float(q[u].x), (int)q[u].y, bv, bi);
    }
    for (; s < slots; s += kArgmaxLanes) {
      const uint2 q = __ldg(part + s * R + row);
      argmax_take(__uint_as_float(q.x), (int)q.y, bv, bi);
    }
  }
  sv[sl][rr] = bv; si[sl][rr] = bi;
  __syncthreads();
  if (sl == 0 && row < R) {
    for (int w = 1; w < kArgmaxLanes; ++w) argmax_take(sv[w][rr], si[w][rr], bv, bi);
    if (bi < 0 || bi >= V) bi = 0;       // all-NaN row
    write_token(out, row, bi);
  }
}

// ---- Philox4x32-10 (Salmon et al., SC'11) ---------------------------------------------------
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

// order-preserving map float -> uint32 (larger float, larger key) and back
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// ---- candidate threshold carried from one selection of a row to its next (fused top-k) ----------
// The LM head with fused top-k keeps, per row, every logit at or above a threshold; the selection is exact when
// that set holds at least k logits. The threshold for the NEXT step of the same sample is taken from this
// step's sorted candidates so that about topk_target(k) logits are expected above it: the logits of consecutive
// positions of one sample have nearly the same scale. With fewer candidates than the target the upper tail is
// continued below the lowest one as an exponential in the value. 0 (all bits zero) stands for "no threshold".
__host__ __device__ inline int topk_target(int k) { return 3 * k > 192 ? 3 * k : 192; }
constexpr int kFusedTopkCap = 1024;      // places per row in the candidate lists
constexpr int kFusedTopkMaxK = 160;      // 3 k must stay well below the capacity

__device__ __forceinline__ float cand_value(unsigned long long w) { return key_value(~(uint32_t)(w >> 32)); }

__device__ inline float next_threshold(const unsigned long long* sorted, int c, int k) {
  const int T = topk_target(k);
  float t;
  if (c >= T) {
    t = cand_value(sorted[T - 1]);
  } else {
    // slope of log(rank) against value between rank i (the k-th, or a quarter of the way in when k is small) and
    // the lowest candidate; with too few candidates below rank i, between the first and the k-th instead
    const int i = k > (c + 3) / 4 ? k : (c + 3) / 4;
    const float v1 = cand_value(sorted[0]), vk = cand_value(sorted[k - 1]), vi = cand_value(sorted[i - 1]),
                vn = cand_value(sorted[c - 1]);
    float s = 0.f;
    if (c >= i + (i / 4 > 2 ? i / 4 : 2)) s = (vi - vn) / logf((float)c / (float)i);
    else if (k >= 2) s = (v1 - vk) / logf((float)k);
    t = vn - s * logf((float)T / (float)c);
    if (!(s > 0.f)) t = 0.f;
  }
  if (!(fabsf(t) < INFINITY)) return 0.f;        // NaN, infinities: none
  return t == 0.f ? -0.0f : t;                   // a threshold of zero keeps a bit set
}

// Thread 0 of a block: inverse-CDF draw over the k first of `sorted` (logit desc, id asc) and the row's outputs.
__device__ inline void draw_topk(const unsigned long long* sorted, int c, int k, float inv_temp, uint64_t seed,
                                 uint64_t sidx, int step, const SelectOut& out, int64_t row, float* cdf) {
  const float l0 = cand_value(sorted[0]);
  float acc = 0.f;
  for (int i = 0; i < k; ++i) {
    acc += expf((cand_value(sorted[i]) - l0) * inv_temp);
    cdf[i] = acc;
  }
  const uint32_t r = philox4x32_10_word0((uint32_t)sidx, (uint32_t)(out.ctr != nullptr ? out.ctr[kCtrStep] : step), 0u, 0u,
                                         (uint32_t)seed, (uint32_t)(seed >> 32));
  const float u = (float)(r >> 8) * (1.0f / 16777216.0f);
  const float target = u * acc;
  int pick = k - 1;
  for (int i = 0; i < k; ++i) {
    if (cdf[i] > target) { pick = i; break; }
  }
  if (out.thr_out != nullptr) out.thr_out[row] = next_threshold(sorted, c, k);
  write_token(out, row, (int)(uint32_t)(sorted[pick] & 0xffffffffull));
}

// Sorts cand[0 .. c) of a block's shared memory ascending, i.e. by (logit desc, id asc); c <= the array's
// power-of-two capacity. All threads of the block call it.
__device__ inline void sort_candidates(unsigned long long* cand, int c, int tid, int nthreads) {
  int P = 2;
  while (P < c) P <<= 1;
  for (int i = c + tid; i < P; i += nthreads) cand[i] = ~0ull;
  __syncthreads();
  for (int size = 2; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < P; i += nthreads) {
        const int j = i ^ stride;
        if (j > i) {
          const unsigned long long a = cand[i], b = cand[j];
          const bool up = (i & size) == 0;
          if ((a > b) == up) { cand[i] = b; cand[j] = a; }
        }
      }
      __syncthreads();
    }
  }
}

// ---- top-k + temperature + inverse-CDF draw ------------------------------------------------
// 1. radix-select (4 passes of 8 bits) the key of the k-th largest logit;
// 2. collect everything above it, plus the lowest ids among the ties at it;
// 3. bitonic-sort the <= 256 candidates by (logit desc, id asc);
// 4. one thread accumulates w_i = exp((l_i - l_0)/T) in that order and picks the first
//    cumulative weight exceeding u * total.
template <bool ROW_IN_SMEM>
__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(const float* __restrict__ logits, int64_t R, int V, int k, float inv_temp, uint64_t seed,
                   uint64_t sample_base, int step, SelectOut out, uint32_t* status, int only_marked) {
  pdl_trigger();
  pdl_wait();
  int64_t row, lrow;
  if (!select_rows(out, blockIdx.x, R, &row, &lrow)) return;
  // second stage of the streaming kernel below: only the rows it marked (-1) are processed here
  if (only_marked && out.last_tok[row] != -1) return;
  extern __shared__ float srow[];
  __shared__ uint32_t hist[256];
  __shared__ unsigned long long cand[kTopKMax];
  __shared__ uint32_t sh_prefix, sh_need, sh_ties, sh_count, sh_running;
  __shared__ uint32_t warp_cnt[kSelThreads / 32];

  const float* lr = logits + lrow * (int64_t)V;
  const int tid = threadIdx.x;
  bool bad = false;
  if (ROW_IN_SMEM) {
    for (int i = tid * 4; i < V; i += kSelThreads * 4) {
      const float4 v = *reinterpret_cast<const float4*>(lr + i);
      bad |= !(v.x == v.x) | !(v.y == v.y) | !(v.z == v.z) | !(v.w == v.w);
      *reinterpret_cast<float4*>(srow + i) = v;
    }
  }
  if (bad) raise_status(status, kStatusNonFinite);
  const float* src = ROW_IN_SMEM ? srow : lr;
  if (tid == 0) { sh_prefix = 0; sh_need = (uint32_t)k; sh_count = 0; sh_running = 0; }
  __syncthreads();

  uint32_t mask = 0;
  for (int shift = 24; shift >= 0; shift -= 8) {
    hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = sh_prefix;
    for (int i = tid; i < V; i += kSelThreads) {
      const uint32_t key = order_key(src[i]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t need = sh_need, cum = 0;
      int digit = 0;
      for (int b = 255; b >= 0; --b) {
        if (cum + hist[b] >= need) { digit = b; break; }
        cum += hist[b];
      }
      sh_need = need - cum;              // how many still to take inside this digit
      sh_prefix = prefix | ((uint32_t)digit << shift);
      sh_ties = hist[digit];             // after the last pass: number of keys equal to the threshold
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t thr = sh_prefix, need_ties = sh_need, ties = sh_ties;
  const uint32_t n_above = (uint32_t)k - need_ties;

  // keys strictly above the threshold: order does not matter (sorted below)
  for (int i = tid; i < V; i += kSelThreads) {
    const uint32_t key = order_key(src[i]);
    if (key > thr || (key == thr && ties == need_ties)) {
      const uint32_t slot = atomicAdd(&sh_count, 1u);
      if (slot < (uint32_t)kTopKMax) cand[slot] = ((unsigned long long)(~key) << 32) | (uint32_t)i;
    }
  }
  if (ties != need_ties) {
    // more ties than places: take the lowest ids, found by a block-wide ordered scan
    const int warp = tid >> 5, lane = tid & 31;
    for (int base = 0; base < V; base += kSelThreads) {
      const int i = base + tid;
      const bool f = (i < V) && (order_key(src[i]) == thr);
      const uint32_t bal = __ballot_sync(0xffffffffu, f);
      if (lane == 0) warp_cnt[warp] = __popc(bal);
      __syncthreads();
      uint32_t off = sh_running;
      for (int w = 0; w < warp; ++w) off += warp_cnt[w];
      off += __popc(bal & ((1u << lane) - 1u));
      if (f && off < need_ties) cand[n_above + off] = ((unsigned long long)(~thr) << 32) | (uint32_t)i;
      __syncthreads();
      if (tid == 0) {
        uint32_t t = 0;
        for (int w = 0; w < kSelThreads / 32; ++w) t += warp_cnt[w];
        sh_running += t;
      }
      __syncthreads();
      if (sh_running >= need_ties) break;
    }
  }
  __syncthreads();
  // pad to a power of two and sort ascending by (~key, id) = (logit desc, id asc)
  int P = 1;
  while (P < k) P <<= 1;
  if (tid >= k && tid < P) cand[tid] = ~0ull;
  __syncthreads();
  for (int size = 2; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      if (tid < P) {
        const int j = tid ^ stride;
        if (j > tid) {
          const unsigned long long a = cand[tid], b = cand[j];
          const bool up = (tid & size) == 0;
          if ((a > b) == up) { cand[tid] = b; cand[j] = a; }
        }
      }
      __syncthreads();
    }
  }
  if (tid == 0) {
    const float l0 = key_value(~(uint32_t)(cand[0] >> 32));
    float* cdf = reinterpret_cast<float*>(hist);     // reuse: k <= 256 floats
    float c = 0.f;
    for (int i = 0; i < k; ++i) {
      const float li = key_value(~(uint32_t)(cand[i] >> 32));
      c += expf((li - l0) * inv_temp);
      cdf[i] = c;
    }
    const uint64_t sidx = sample_base + (uint64_t)row;
    const uint32_t r = philox4x32_10_word0((uint32_t)sidx, (uint32_t)(out.ctr != nullptr ? out.ctr[kCtrStep] : step), 0u, 0u, (uint32_t)seed,
                                           (uint32_t)(seed >> 32));
    const float u = (float)(r >> 8) * (1.0f / 16777216.0f);
    const float target = u * c;
    int pick = k - 1;
    for (int i = 0; i < k; ++i) {
      if (cdf[i] > target) { pick = i; break; }
    }
    if (out.thr_out != nullptr) out.thr_out[row] = 0.f;     // no candidate set to take a threshold from
    write_token(out, row, (int)(uint32_t)(cand[pick] & 0xffffffffull));
  }
}

// ---- top-k, streaming version ------------------------------------------------------------------
// The radix selection above makes four histogram passes over a row held in shared memory; with logits
// that share their leading bits almost all of its shared-memory atomics land in one or two bins. This
// kernel instead (1) streams the row once for mean and standard deviation, (2) streams it again (an L2
// hit) collecting every logit >= t = mean + z * sd, and accepts the candidate set when it holds at least
// k and at most kTopkCap entries: any set {x >= t} with >= k members contains the k largest logits and all
// ties at the k-th place, so sorting it by (logit desc, id asc) gives exactly the order the radix version
// gives. z starts at the normal quantile for an expected 2.5 k candidates (z0, from the host) and is
// bisected when the count misses the window. Rows that still miss it after kTopkRounds (constant rows,
// infinities, more than kTopkCap ties) are marked with token -1 and redone by select_topk_kernel.
// Little shared memory, so several rows are in flight per SM and the row never has to fit on chip.
constexpr int kTopkCap = 1024;
constexpr int kTopkRounds = 6;

__global__ void __launch_bounds__(kSelThreads)
select_topk_stream_kernel(const float* __restrict__ logits, int64_t R, int V, int k, float inv_temp, float z0,
                          uint64_t seed, uint64_t sample_base, int step, SelectOut out, uint32_t* status) {
  pdl_trigger();
  pdl_wait();
  __shared__ unsigned long long cand[kTopkCap];
  __shared__ float red_s[kSelThreads / 32], red_q[kSelThreads / 32];
  __shared__ float sh_mean, sh_sd;
  __shared__ uint32_t sh_count;
  __shared__ float cdf[kTopKMax];

  int64_t row, lrow;
  if (!select_rows(out, blockIdx.x, R, &row, &lrow)) return;
  const float* lr = logits + lrow * (int64_t)V;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- pass 1: moments ----
  float sum = 0.f, sq = 0.f;
  bool bad = false;
  for (int i = tid * 4; i < V; i += kSelThreads * 4) {
    const float4 v = *reinterpret_cast<const float4*>(lr + i);
    bad |= !(v.x == v.x) | !(v.y == v.y) | !(v.z == v.z) | !(v.w == v.w);
    sum += (v.x + v.y) + (v.z + v.w);
    sq = fmaf(v.x, v.x, sq); sq = fmaf(v.y, v.y, sq); sq = fmaf(v.z, v.z, sq); sq = fmaf(v.w, v.w, sq);
  }
  if (bad) raise_status(status, kStatusNonFinite);
  sum = warp_sum(sum); sq = warp_sum(sq);
  if (lane == 0) { red_s[warp] = sum; red_q[warp] = sq; }
  __syncthreads();
  if (tid == 0) {
    float a = 0.f, b = 0.f;
    for (int w = 0; w < kSelThreads / 32; ++w) { a += red_s[w]; b += red_q[w]; }
    const float mean = a / (float)V;
    sh_mean = mean;
    sh_sd = sqrtf(fmaxf(b / (float)V - mean * mean, 0.f));
    sh_count = 0;
  }
  __syncthreads();
  const float mean = sh_mean, sd = sh_sd;

  // ---- pass 2 (repeated while the count misses [k, kTopkCap]): collect everything >= t ----
  float z = z0, lo = -INFINITY, hi = INFINITY;       // lo: a z that gave too many, hi: one that gave too few
  uint32_t c = 0;
  bool found = false;
  for (int round = 0; round < kTopkRounds; ++round) {
    const float t = fmaf(z, sd, mean);
    for (int i = tid * 4; i < V; i += kSelThreads * 4) {
      const float4 v = *reinterpret_cast<const float4*>(lr + i);
      const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (e[j] >= t) {
          const uint32_t slot = atomicAdd(&sh_count, 1u);
          if (slot < (uint32_t)kTopkCap) cand[slot] = ((unsigned long long)(~order_key(e[j])) << 32) | (uint32_t)(i + j);
        }
      }
    }
    __syncthreads();
    c = sh_count;
    __syncthreads();
    if (c >= (uint32_t)k && c <= (uint32_t)kTopkCap) { found = true; break; }
    if (tid == 0) sh_count = 0;
    if (c < (uint32_t)k) hi = z; else lo = z;
    z = (lo > -INFINITY && hi < INFINITY) ? 0.5f * (lo + hi) : (c < (uint32_t)k ? z - 1.0f : z + 0.75f);
    __syncthreads();
  }
  if (!found) {                                      // block-uniform
    if (tid == 0) out.last_tok[row] = -1;
    return;
  }

  sort_candidates(cand, (int)c, tid, kSelThreads);
  if (tid == 0) draw_topk(cand, (int)c, k, inv_temp, seed, sample_base + (uint64_t)row, step, out, row, cdf);
}

// ---- top-k fused into the LM head: second stage ------------------------------------------------------
// The LM head (kEpiCollect epilogue) has left, per row, the logits at or above the row's threshold as sortable
// words in lists[row][0 .. cnt[row]). A row whose list holds at least k and at most `cap` of them is settled
// here exactly as the streaming kernel settles it (any set {x >= t} with at least k members contains the k
// largest logits and every tie at the k-th place): sort, softmax weights, Philox draw. A row without a
// threshold yet, with fewer than k candidates, or with more than fit is handed back: its activation row is
// copied to the next free row of a_fb and its index to fb_rows (n_fb counts them), and the caller recomputes
// the logits of just those rows and runs the streaming kernel on them (SelectOut::row_map).
__global__ void __launch_bounds__(kSelThreads)
topk_merge_kernel(const unsigned long long* __restrict__ lists, const uint32_t* __restrict__ cnt, const float* __restrict__ thr,
                  int cap, int64_t R, int k, float inv_temp, uint64_t seed, uint64_t sample_base, int step, SelectOut out,
                  const uint4* __restrict__ a, uint4* __restrict__ a_fb, int row_vecs, int32_t* __restrict__ fb_rows,
                  uint32_t* __restrict__ n_fb, uint32_t* __restrict__ handed_back) {
  pdl_trigger();
  pdl_wait();
  __shared__ unsigned long long cand[kFusedTopkCap];
  __shared__ float cdf[kTopKMax];
  __shared__ uint32_t sh_idx;
  const int64_t row = blockIdx.x;
  if (row >= R) return;
  const int tid = threadIdx.x;
  const uint32_t c = cnt[row];
  const float t = thr[row];
  const bool have_thr = (t == t) && __float_as_uint(t) != 0u;
  if (!have_thr || c < (uint32_t)k || c > (uint32_t)cap) {          // block-uniform
    if (tid == 0) {
      const uint32_t idx = atomicAdd(n_fb, 1u);
      fb_rows[idx] = (int32_t)row;
      sh_idx = idx;
      if (handed_back != nullptr) atomicAdd(handed_back, 1u);
    }
    __syncthreads();
    const uint4* src = a + row * (int64_t)row_vecs;
    uint4* dst = a_fb + (int64_t)sh_idx * row_vecs;
    for (int i = tid; i < row_vecs; i += kSelThreads) dst[i] = src[i];
    return;
  }
  const unsigned long long* lr = lists + row * (int64_t)cap;
  for (int i = tid; i < (int)c; i += kSelThreads) cand[i] = lr[i];
  __syncthreads();
  sort_candidates(cand, (int)c, tid, kSelThreads);
  if (tid == 0) draw_topk(cand, (int)c, k, inv_temp, seed, sample_base + (uint64_t)row, step, out, row, cdf);
}

// Cache rows of `replicas` consecutive samples = the row of their prompt:
// dst[(p0 + p) * replicas + j, :] = src[p, :] for p < np, j < replicas (16-byte vectors; one layer).
__global__ void __launch_bounds__(256)
broadcast_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int64_t np, int64_t replicas, int64_t vec_per_row) {
  pdl_trigger();
  pdl_wait();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= np * replicas * vec_per_row) return;
  const int64_t row = i / vec_per_row, v = i % vec_per_row;
  dst[i] = __ldg(src + (row / replicas) * vec_per_row + v);
}

// Per-sample positions after a prefill of prompts of different lengths: the lengths as the prefill used them
// (clamped to [1, n_max]), so that the decode steps continue from the same positions.
__global__ void __launch_bounds__(256)
clamp_lengths_kernel(const int32_t* __restrict__ len, int32_t* __restrict__ pos, int64_t B, int lo, int hi) {
  pdl_trigger();
  pdl_wait();
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i < B) pos[i] = min(max(len[i], lo), hi);
}

// Step counters in the state header: set before a replayed generation loop, advanced after every step.
__global__ void set_counters_kernel(int32_t* hdr, int pos, int step, int col) {
  pdl_trigger();
  pdl_wait();
  hdr[kCtrPos] = pos; hdr[kCtrStep] = step; hdr[kCtrCol] = col;
}
__global__ void advance_counters_kernel(int32_t* hdr) {
  pdl_trigger();
  pdl_wait();
  hdr[kCtrPos] += 1; hdr[kCtrStep] += 1; hdr[kCtrCol] += 1;
}

}  // namespace srm
