// Work lists of the fused feed-forward kernel (ffn_fused.cuh): which CTA pair computes which 256 x 256 tile of the
// up projection H = gelu(a W1^T + b1) and of the down projection x += H W2^T + b2, and in which order.
// Plain host C++ (no CUDA): the plan is made on the host and travels to the kernel as a launch parameter.
//
// A down tile of row block rb reads H[rb, :] k-block by k-block, so it may START before the up tiles of its row
// block are finished: it needs column tile hc of H only when its k-loop gets there. The plan uses this to end all
// pairs together although the down tiles are few and long (mid model, 4096 rows: 64 tiles of 64 k-blocks for 74
// pairs): some pairs compute up tiles to the end while the others already run down tiles that consume those up
// tiles as they appear.
//
// The plan is found by list scheduling in REVERSED time. Seen backwards, a down tile has no predecessor, and an
// up tile (rb, hc) is released once every down tile of rb has been running long enough (backwards) to be past
// column tile hc; with release times instead of predecessors, "never leave a pair idle while something is
// released" is a good rule, and all down tiles of the last row blocks start together at reversed time 0, i.e. end
// together. Turning each pair's list around gives the forward lists. Every dependency of the forward lists points
// from an item that ends earlier in model time to one that ends later, so the lists can never deadlock, whatever
// the real durations are (ffn_simulate() re-checks that by running them forward).
#pragma once

#include <stdint.h>

#include <algorithm>
#include <vector>

#ifdef __CUDACC__
#define SRM_HD __host__ __device__
#else
#define SRM_HD
#endif

namespace srm {
namespace tc {

constexpr int kFfnMaxItems = 2048;     // tiles of both projections in one launch
constexpr int kFfnMaxPairs = 96;
constexpr int kFfnMaxRb = 64;          // row blocks of 256 rows
constexpr int kFfnMaxCu = 32;          // column tiles of H (F <= 8192)
constexpr int kFfnKbPerHTile = 4;      // k-blocks (64) of the down projection per column tile (256) of H

// Item: bit 15 = down projection, bits 5..10 = row block, bits 0..4 = column tile; up projection only: bit 14 = one
// 256 x 128 half of the tile (the tiles of a last, partly filled round of up tiles run as two halves on two pairs,
// which ends earlier than whole tiles on half as many pairs), bit 13 = its second half (columns 128..255).
struct FfnPlan {
  uint16_t n_pairs;
  uint16_t off[kFfnMaxPairs + 1];      // pair c owns item[off[c]] .. item[off[c + 1] - 1], in order
  uint16_t item[kFfnMaxItems];
};
SRM_HD inline uint16_t ffn_item(bool down, int rb, int cb) { return (uint16_t)((down ? 0x8000 : 0) | (rb << 5) | cb); }
SRM_HD inline bool ffn_item_down(uint16_t it) { return (it & 0x8000) != 0; }
SRM_HD inline int ffn_item_rb(uint16_t it) { return (it >> 5) & 63; }
SRM_HD inline int ffn_item_cb(uint16_t it) { return it & 31; }
SRM_HD inline bool ffn_item_half(uint16_t it) { return (it & 0x4000) != 0; }
SRM_HD inline int ffn_item_noff(uint16_t it) { return (it & 0x2000) ? 128 : 0; }     // first column inside the tile
constexpr uint16_t kFfnHalf = 0x4000, kFfnSecond = 0x2000;
constexpr double kFfnHalfCost = 0.75;  // a half piece moves three quarters of a tile's operand bytes for half its flops

struct FfnShape {
  int Rb;        // row blocks
  int Cu, ku;    // up projection: column tiles (F / 256), k-blocks per tile (d / 64)
  int Cd, kd;    // down projection: column tiles (d / 256), k-blocks per tile (F / 64 = 4 Cu)
};

// Cost model, in units of one k-block of the LM head's main loop (about 640 clock cycles, 0.38 us). From device
// timestamps of this kernel on the mid model (4096 rows): an up tile of 16 k-blocks takes 7.25 us (its epilogue
// stages and stores 128 KB beside the next tile's main loop), a down tile of 64 k-blocks 24 us when it never waits,
// and a down tile can multiply a column tile of H 6.3 us after the up tile's last MMA has completed (GELU epilogue of
// 16 warps, bulk stores, counter, load) - a lag that decides how late the last up tiles may be placed.
struct FfnCost {
  double up_kb = 1.0, up_tile = 3.1, dn_kb = 0.96, dn_tile = 1.5, ready_lag = 16.5;
  double h_budget_bytes = 48.0 * 1024 * 1024;   // H of the row blocks whose down tiles are under way but whose up tiles are not all placed
};

inline bool ffn_shape_ok(const FfnShape& s, int pairs) {
  return s.Rb >= 1 && s.Rb <= kFfnMaxRb && s.Cu >= 1 && s.Cu <= kFfnMaxCu && s.Cd >= 1 && s.Cd <= 8 && s.ku >= 1 &&
         s.kd == kFfnKbPerHTile * s.Cu && pairs >= 1 && pairs <= kFfnMaxPairs && s.Rb * (s.Cu + s.Cd) + kFfnMaxPairs / 2 <= kFfnMaxItems;
}

// Forward run of a plan under the cost model. Returns the time the last pair ends, or -1 when the lists block one
// another (never for a plan of ffn_make_plan) or do not hold every tile exactly once.
inline double ffn_simulate(const FfnShape& s, const FfnPlan& P, const FfnCost& c = FfnCost()) {
  const int n = P.n_pairs;
  std::vector<double> ready((size_t)s.Rb * s.Cu, -1.0);      // time H tile (rb, hc) becomes visible; -1: not known yet
  std::vector<int> seen_up((size_t)s.Rb * s.Cu, 0), seen_dn((size_t)s.Rb * s.Cd, 0);
  std::vector<double> pend((size_t)s.Rb * s.Cu, 0.0);        // end of the first half of a tile computed in halves
  std::vector<int> pos(n, 0);
  std::vector<double> t(n, 0.0);
  int left = 0, halves = 0;
  for (int p = 0; p < n; ++p) {
    if (P.off[p + 1] < P.off[p] || P.off[p + 1] > kFfnMaxItems) return -1.0;
    left += P.off[p + 1] - P.off[p];
    for (int i = P.off[p]; i < P.off[p + 1]; ++i) halves += ffn_item_half(P.item[i]) ? 1 : 0;
  }
  if (halves % 2 || left - halves / 2 != s.Rb * (s.Cu + s.Cd)) return -1.0;
  bool progress = true;
  while (left > 0 && progress) {
    progress = false;
    for (int p = 0; p < n; ++p) {
      while (P.off[p] + pos[p] < P.off[p + 1]) {
        const uint16_t it = P.item[P.off[p] + pos[p]];
        const int rb = ffn_item_rb(it), cb = ffn_item_cb(it);
        if (rb >= s.Rb) return -1.0;
        if (!ffn_item_down(it)) {
          // seen_up: bit 0 = columns 0..127 computed, bit 1 = columns 128..255
          if (cb >= s.Cu) return -1.0;
          int& seen = seen_up[(size_t)rb * s.Cu + cb];
          const int bits = ffn_item_half(it) ? (ffn_item_noff(it) ? 2 : 1) : 3;
          if (seen & bits) return -1.0;
          seen |= bits;
          t[p] += (ffn_item_half(it) ? kFfnHalfCost : 1.0) * s.ku * c.up_kb + c.up_tile;
          if (seen == 3) ready[(size_t)rb * s.Cu + cb] = std::max(pend[(size_t)rb * s.Cu + cb], t[p]) + c.ready_lag;
          else pend[(size_t)rb * s.Cu + cb] = t[p];
        } else {
          if (cb >= s.Cd) return -1.0;
          bool known = true;
          for (int hc = 0; hc < s.Cu; ++hc) known = known && ready[(size_t)rb * s.Cu + hc] >= 0.0;
          if (!known) break;                                   // this pair waits for tiles no pair has reached yet
          if (seen_dn[(size_t)rb * s.Cd + cb]++) return -1.0;
          double u = t[p] + c.dn_tile;
          for (int hc = 0; hc < s.Cu; ++hc) u = std::max(u, ready[(size_t)rb * s.Cu + hc]) + kFfnKbPerHTile * c.dn_kb;
          t[p] = u;
        }
        ++pos[p];
        --left;
        progress = true;
      }
    }
  }
  if (left > 0) return -1.0;
  double end = 0.0;
  for (int p = 0; p < n; ++p) end = std::max(end, t[p]);
  return end;
}

// Lower bound of any plan under the cost model: all work shared out evenly, and at least one up and one down tile in a row.
inline double ffn_ideal(const FfnShape& s, int pairs, const FfnCost& c = FfnCost()) {
  const double up = s.ku * c.up_kb + c.up_tile, dn = s.kd * c.dn_kb + c.dn_tile;
  return std::max(((double)s.Rb * s.Cu * up + (double)s.Rb * s.Cd * dn) / pairs, up + kFfnKbPerHTile * c.dn_kb + dn);
}

// The plan in which the last `n_half` up tiles placed (the first of the forward lists) go out as halves.
inline bool ffn_make_plan_halves(const FfnShape& s, int pairs, int n_half, FfnPlan* out, const FfnCost& c) {
  if (!ffn_shape_ok(s, pairs)) return false;
  const double up_cost = s.ku * c.up_kb + c.up_tile, dn_cost = s.kd * c.dn_kb + c.dn_tile;
  const double h_tile = kFfnKbPerHTile * c.dn_kb;             // time a down tile spends on one column tile of H
  const double rb_bytes = 256.0 * 256.0 * s.Cu * 2.0;
  const int open_max = std::max(2, (int)(c.h_budget_bytes / rb_bytes));

  std::vector<double> free_at(pairs, 0.0);
  std::vector<std::vector<uint16_t>> rev(pairs);              // items in reversed time order
  // per row block: down tiles placed so far, the latest reversed start among them, up tiles placed so far
  std::vector<int> dn_placed(s.Rb, 0), up_placed(s.Rb, 0);
  std::vector<double> dn_start(s.Rb, 0.0);
  int next_dn_rb = s.Rb - 1;                                  // down tiles go from the last row block to the first
  int open = 0;                                               // row blocks with a down tile placed and up tiles left
  int left = s.Rb * (s.Cu + s.Cd);
  int ups_left = s.Rb * s.Cu, dns_left = s.Rb * s.Cd;
  int pending_half = -1;                                      // the second half of a tile whose first half has been placed
  double pending_rel = 0.0;
  const double half_cost = kFfnHalfCost * s.ku * c.up_kb + c.up_tile;
  while (left > 0) {
    int p = 0;
    for (int q = 1; q < pairs; ++q) if (free_at[q] < free_at[p]) p = q;
    const double t = free_at[p];
    if (pending_half >= 0) {                                  // (goes to the next pair that is free, whatever else is released)
      rev[p].push_back((uint16_t)pending_half);
      free_at[p] = std::max(t, pending_rel) + half_cost;
      pending_half = -1;
      --left;
      continue;
    }
    // (a) a down tile: of a row block already begun, or of the next one while the H budget allows
    while (next_dn_rb >= 0 && dn_placed[next_dn_rb] == s.Cd) --next_dn_rb;
    const bool dn_ok = next_dn_rb >= 0 && (dn_placed[next_dn_rb] > 0 || open < open_max);
    if (dn_ok) {
      const int rb = next_dn_rb;
      if (dn_placed[rb] == 0) ++open;
      rev[p].push_back(ffn_item(true, rb, s.Cd - 1 - dn_placed[rb]));
      dn_start[rb] = std::max(dn_start[rb], t);
      ++dn_placed[rb];
      free_at[p] = t + dn_cost;
      --left;
      --dns_left;
      continue;
    }
    // (b) a released up tile: the highest row block first, within it the highest column tile (placed backwards)
    int best_rb = -1;
    double soonest = -1.0;                                    // earliest release among the tiles not yet released
    for (int rb = s.Rb - 1; rb >= 0; --rb) {
      if (dn_placed[rb] < s.Cd || up_placed[rb] == s.Cu) continue;
      const int hc = s.Cu - 1 - up_placed[rb];
      const double rel = dn_start[rb] + (s.Cu - hc) * h_tile + c.ready_lag;
      if (rel <= t) { best_rb = rb; break; }
      if (soonest < 0.0 || rel < soonest) soonest = rel;
    }
    if (best_rb >= 0) {
      const int rb = best_rb, hc = s.Cu - 1 - up_placed[rb];
      // the last up tiles (in reversed time: the first of the forward lists), when they no longer fill a round of
      // whole tiles, go out as halves to twice as many pairs
      const bool halves = dns_left == 0 && ups_left <= n_half;
      if (halves) {
        rev[p].push_back((uint16_t)(ffn_item(false, rb, hc) | kFfnHalf | kFfnSecond));
        pending_half = ffn_item(false, rb, hc) | kFfnHalf;
        pending_rel = t;
        ++left;                                               // one tile, two items
        free_at[p] = t + half_cost;
      } else {
        rev[p].push_back(ffn_item(false, rb, hc));
        free_at[p] = t + up_cost;
      }
      if (++up_placed[rb] == s.Cu) --open;
      --ups_left;
      --left;
      continue;
    }
    // nothing released for this pair now: it idles until the next release (or until another pair frees up and
    // places the down tiles that release more)
    double wake = soonest;
    for (int q = 0; q < pairs; ++q) if (free_at[q] > t && (wake < 0.0 || free_at[q] < wake)) wake = free_at[q];
    if (wake <= t) return false;                              // cannot happen: something is always pending
    free_at[p] = wake;
  }
  out->n_pairs = (uint16_t)pairs;
  int o = 0;
  for (int p = 0; p < pairs; ++p) {
    out->off[p] = (uint16_t)o;
    for (auto it = rev[p].rbegin(); it != rev[p].rend(); ++it) out->item[o++] = *it;
  }
  for (int p = pairs; p <= kFfnMaxPairs; ++p) out->off[p] = (uint16_t)o;
  return ffn_simulate(s, *out, c) >= 0.0;
}

// The plan of the decode step: as few up tiles in halves as reach (within half a k-block time) the shortest plan any
// number of halves up to pairs / 2 gives. A half moves three quarters of a tile's operand bytes for half its flops,
// and the step runs at the power cap: halves that do not shorten the plan only cost clock.
inline bool ffn_make_plan(const FfnShape& s, int pairs, FfnPlan* out, const FfnCost& c = FfnCost()) {
  if (!ffn_shape_ok(s, pairs)) return false;
  const int h_max = std::min(pairs / 2, s.Rb * s.Cu);
  std::vector<double> len(h_max + 1, -1.0);
  double best = -1.0;
  for (int h = 0; h <= h_max; ++h) {
    if (!ffn_make_plan_halves(s, pairs, h, out, c)) continue;
    len[h] = ffn_simulate(s, *out, c);
    if (len[h] >= 0.0 && (best < 0.0 || len[h] < best)) best = len[h];
  }
  if (best < 0.0) return false;
  for (int h = 0; h <= h_max; ++h)
    if (len[h] >= 0.0 && len[h] <= best + 0.5) return ffn_make_plan_halves(s, pairs, h, out, c);
  return false;
}

}  // namespace tc
}  // namespace srm
