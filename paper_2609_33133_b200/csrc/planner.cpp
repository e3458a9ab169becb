// Replay-grid assignment (Sec. 3.4 "Replay units and grid assignment", Eq. 6): host only.
//
// U units with work w_k and size m_k go onto a grid of b rounds x s lanes.  Lanes of a round
// run side by side and rounds one after the other, so the predicted critical path is the sum
// over rounds of the heaviest lane of the round; a (round, lane) cell holds at most `cap` of
// size.  Up to `exact_max_units` units the minimum is found exactly by dynamic programming
// over subsets (the paper's bounded AssignGrid); above it units are placed largest first.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <map>
#include <numeric>
#include <vector>

#include "../../include/augtree.h"

namespace {

constexpr int64_t kInf = std::numeric_limits<int64_t>::max() / 4;
constexpr int kHardMaxExact = 16;  // 3^16 subset pairs is the most the exact solver is allowed

// Exact solver.  lane_best[j][S]: least possible heaviest lane when the units of S share j lanes
// of one round (kInf if they do not fit); round_best[t][S]: least path when S is spread over t rounds.
// Both recurrences peel off the part that contains the lowest unit of S, which visits every
// partition once.
struct ExactGrid {
  int U, b, s;
  std::vector<int64_t> wsum, msum;
  std::vector<std::vector<int64_t>> lane_best, round_best;
  std::vector<std::vector<uint32_t>> lane_pick, round_pick;

  bool solve(const int64_t *w, const int64_t *m, int64_t cap) {
    const uint32_t full = (1u << U) - 1;
    wsum.assign(full + 1, 0);
    msum.assign(full + 1, 0);
    for (uint32_t S = 1; S <= full; ++S) {
      const int k = __builtin_ctz(S);
      wsum[S] = wsum[S & (S - 1)] + w[k];
      msum[S] = msum[S & (S - 1)] + (m ? m[k] : 0);
    }
    auto fits = [&](uint32_t T) { return cap <= 0 || msum[T] <= cap; };
    lane_best.assign(s + 1, std::vector<int64_t>(full + 1, kInf));
    lane_pick.assign(s + 1, std::vector<uint32_t>(full + 1, 0));
    for (int j = 0; j <= s; ++j) lane_best[j][0] = 0;
    for (int j = 1; j <= s; ++j)
      for (uint32_t S = 1; S <= full; ++S) {
        const uint32_t low = S & (~S + 1), rest = S ^ low;
        // T = low | (any subset of rest): the lane that takes the lowest unit
        for (uint32_t sub = rest;; sub = (sub - 1) & rest) {
          const uint32_t T = sub | low;
          if (fits(T) && lane_best[j - 1][S ^ T] < kInf) {
            const int64_t v = std::max(wsum[T], lane_best[j - 1][S ^ T]);
            if (v < lane_best[j][S]) { lane_best[j][S] = v; lane_pick[j][S] = T; }
          }
          if (sub == 0) break;
        }
      }
    round_best.assign(b + 1, std::vector<int64_t>(full + 1, kInf));
    round_pick.assign(b + 1, std::vector<uint32_t>(full + 1, 0));
    for (int t = 0; t <= b; ++t) round_best[t][0] = 0;
    for (int t = 1; t <= b; ++t)
      for (uint32_t S = 1; S <= full; ++S) {
        const uint32_t low = S & (~S + 1), rest = S ^ low;
        for (uint32_t sub = rest;; sub = (sub - 1) & rest) {
          const uint32_t T = sub | low;
          if (lane_best[s][T] < kInf && round_best[t - 1][S ^ T] < kInf) {
            const int64_t v = lane_best[s][T] + round_best[t - 1][S ^ T];
            if (v < round_best[t][S]) { round_best[t][S] = v; round_pick[t][S] = T; }
          }
          if (sub == 0) break;
        }
      }
    return round_best[b][full] < kInf;
  }

  // placement that attains round_best[rounds][all units] (rounds <= b)
  void unpack(int32_t *round_out, int32_t *lane_out, int rounds = -1) const {
    uint32_t S = (1u << U) - 1;
    int t = rounds < 0 ? b : rounds, round = 0;
    while (S) {
      const uint32_t R = round_pick[t][S];
      uint32_t L = R;
      int j = s, lane = 0;
      while (L) {
        const uint32_t T = lane_pick[j][L];
        for (uint32_t x = T; x; x &= x - 1) {
          const int k = __builtin_ctz(x);
          round_out[k] = round;
          lane_out[k] = lane;
        }
        L ^= T; --j; ++lane;
      }
      S ^= R; --t; ++round;
    }
  }
};

}  // namespace

static int assign_grid_impl(const int64_t *weight, const int64_t *size, int n_units, int n_rounds, int n_lanes,
                            int64_t cell_cap, int exact_max_units, int32_t *round_out, int32_t *lane_out,
                            int64_t *critical_path, int32_t *solved_exactly) {
  if (n_units < 0 || n_rounds < 1 || n_lanes < 1 || (n_units > 0 && (!weight || !round_out || !lane_out))) return AUGTREE_ERR_INVALID_ARG;
  if (cell_cap > 0 && !size && n_units > 0) return AUGTREE_ERR_INVALID_ARG;
  if (n_rounds > 1024 || n_lanes > 65536) return AUGTREE_ERR_UNSUPPORTED;
  for (int k = 0; k < n_units; ++k)
    if (weight[k] < 0 || (size && size[k] < 0) || weight[k] > kInf / (n_units + 1)) return AUGTREE_ERR_INVALID_ARG;
  if (exact_max_units <= 0) exact_max_units = 12;
  exact_max_units = std::min(exact_max_units, kHardMaxExact);
  int64_t path = 0;
  bool exact = false;
  if (n_units == 0) {
    exact = true;
  } else if (n_units <= exact_max_units) {
    ExactGrid g;
    g.U = n_units; g.b = n_rounds; g.s = n_lanes;
    // more lanes (rounds) than units cannot help: cap them so that the tables stay small
    g.s = std::min(g.s, n_units);
    g.b = std::min(g.b, n_units);
    if (!g.solve(weight, size, cell_cap)) return AUGTREE_ERR_UNSUPPORTED;  // the units do not fit the grid
    g.unpack(round_out, lane_out);
    path = g.round_best[g.b][(1u << n_units) - 1];
    exact = true;
  } else {
    // largest first; each unit to the cell that fits and lengthens the path least, then to the lightest
    // such cell, then the lowest round, then the lowest lane
    std::vector<int32_t> ids(n_units);
    std::iota(ids.begin(), ids.end(), 0);
    std::stable_sort(ids.begin(), ids.end(), [&](int32_t a, int32_t c) { return weight[a] > weight[c]; });
    // Empty cells of a round are interchangeable and the lowest lane wins ties, so the occupied lanes of a
    // round are always a prefix 0 .. filled-1: only those and the first empty one are candidates, and only
    // those are stored (the grid itself may be far larger than the number of units).
    std::vector<std::vector<int64_t>> load(n_rounds), used(n_rounds);
    std::vector<int64_t> peak(n_rounds, 0);
    for (int32_t k : ids) {
      int bt = -1, bj = -1;
      int64_t b_grow = 0, b_new = 0;
      for (int t = 0; t < n_rounds; ++t) {
        const int filled = (int)load[t].size();
        for (int j = 0; j < std::min(filled + 1, n_lanes); ++j) {
          const int64_t have = j < filled ? load[t][j] : 0, mem = j < filled ? used[t][j] : 0;
          if (cell_cap > 0 && mem + size[k] > cell_cap) continue;
          const int64_t nw = have + weight[k], grow = std::max(peak[t], nw) - peak[t];
          if (bt < 0 || grow < b_grow || (grow == b_grow && nw < b_new)) { bt = t; bj = j; b_grow = grow; b_new = nw; }
        }
      }
      if (bt < 0) return AUGTREE_ERR_UNSUPPORTED;
      if (bj == (int)load[bt].size()) { load[bt].push_back(0); used[bt].push_back(0); }
      load[bt][bj] += weight[k];
      if (size) used[bt][bj] += size[k];
      peak[bt] = std::max(peak[bt], load[bt][bj]);
      round_out[k] = bt;
      lane_out[k] = bj;
    }
    for (int t = 0; t < n_rounds; ++t) path += peak[t];
  }
  if (critical_path) *critical_path = path;
  if (solved_exactly) *solved_exactly = exact ? 1 : 0;
  return AUGTREE_OK;
}

// Nothing may leave through the C interface but a status code: a failed allocation inside the solvers
// (std::bad_alloc) is reported as AUGTREE_ERR_INTERNAL.
extern "C" int augtree_assign_grid(const int64_t *weight, const int64_t *size, int n_units, int n_rounds, int n_lanes,
                                   int64_t cell_cap, int exact_max_units, int32_t *round_out, int32_t *lane_out,
                                   int64_t *critical_path, int32_t *solved_exactly) {
  try {
    return assign_grid_impl(weight, size, n_units, n_rounds, n_lanes, cell_cap, exact_max_units, round_out, lane_out,
                            critical_path, solved_exactly);
  } catch (...) {
    return AUGTREE_ERR_INTERNAL;
  }
}

// --------------------------------------------------------------------------------------------------------------
// Online strategy planner (Sec. 3.4, Algorithm 1): for one replay tree, enumerate the candidates c = (d, pi, (b, s), X)
// over the given CP degrees, place the replay units (one per response path, weight = valid Q-KV tile count) with
// AssignGrid, score each candidate with Eq. 7-10 and return the cheapest feasible one.  The paper leaves the constants
// of the cost model to profiling: they are inputs.  Readings of what it leaves open (all stated in the header):
// f_ring(d) = (d - 1) / d; lane counts s | d with s <= G; rounds b <= min(b_max, ceil(G / s)); the traffic terms use the
// conservative proxy ceil(G / (b s)) * max_i R_i for the tokens of a cell, so that the placement enters through the
// critical-path work W alone; per-rank memory = prompt share + cell share.
namespace {

constexpr int kTile = 128;
inline int64_t cdiv64(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline double f_ring(int d) { return (double)(d - 1) / (double)d; }
inline int64_t replay_tiles(int64_t P, int64_t R) {
  const int64_t nq = cdiv64(R, kTile);
  return nq * cdiv64(P, kTile) + nq * (nq + 1) / 2;
}
inline int64_t causal_tiles(int64_t n) {
  const int64_t nq = cdiv64(n, kTile);
  return nq * (nq + 1) / 2;
}

}  // namespace

static int plan_tree_impl(const augtree_tree_t *t, const augtree_profile_t *pr, augtree_choice_t *choice, int32_t *round_out,
                          int32_t *lane_out) {
  if (!t || !pr || !choice || t->struct_size != sizeof(augtree_tree_t)) return AUGTREE_ERR_INVALID_ARG;
  const int G = t->n_branches;
  if (t->prompt_len < 1 || G < 0 || (G > 0 && (!t->branch_len || !round_out || !lane_out))) return AUGTREE_ERR_INVALID_ARG;
  if (t->n_degrees < 1 || !t->degrees || t->h_q < 1 || t->h_kv < 1) return AUGTREE_ERR_INVALID_ARG;
  const int b_max = t->b_max > 0 ? t->b_max : 4;
  const int64_t P = t->prompt_len;
  std::vector<int64_t> w(G), m(G);
  int64_t r_max = 0;
  for (int k = 0; k < G; ++k) {
    if (t->branch_len[k] < 1) return AUGTREE_ERR_INVALID_ARG;
    m[k] = t->branch_len[k];
    w[k] = replay_tiles(P, m[k]);
    r_max = std::max(r_max, m[k]);
  }
  bool have = false;
  augtree_choice_t best = {};
  std::vector<int32_t> rounds(G), lanes(G), best_rounds(G), best_lanes(G);
  int n_cand = 0;
  std::map<std::pair<int, int64_t>, ExactGrid> dp_cache;
  for (int di = 0; di < t->n_degrees; ++di) {
    const int d = t->degrees[di];
    if (d < 1 || d > 65536) return AUGTREE_ERR_INVALID_ARG;
    // ---- b = 0: ordinary ring CP over every (P, R_i) pair
    {
      ++n_cand;
      const int64_t longest = P + r_max;
      const bool fits = pr->mem_cap <= 0 || (pr->mem_prompt * (double)P + pr->mem_resp * (double)(longest - P)) / d <= pr->mem_cap;
      if (fits) {
        double total = 0.0;
        for (int k = 0; k < std::max(G, 1); ++k) {
          const int64_t r = G ? m[k] : 0;
          total += pr->alpha_ring * (double)causal_tiles(P + r) / d + pr->beta_ring * 2 * (double)(P + r) * t->h_kv * f_ring(d) +
                   pr->lat_ring0 + pr->lat_ring1 * d;
        }
        const double cost = pr->gamma_ring * total;
        if (!have || cost < best.cost) {
          have = true;
          best.cost = cost; best.degree = d; best.primitive = AUGTREE_RING_CP; best.rounds = 0; best.lanes = 1; best.solved_exactly = 1;
        }
      }
    }
    if (G == 0) continue;
    for (int primitive = AUGTREE_TREE_MOVE_KV; primitive <= AUGTREE_MOVE_Q; ++primitive)
      for (int s = 1; s <= d && s <= G; ++s) {
        if (d % s) continue;
        const int d_lane = d / s;
        // cell limit in response tokens from the per-rank memory model
        int64_t cap = 0;  // 0: none
        if (pr->mem_cap > 0) {
          const double room = primitive == AUGTREE_TREE_MOVE_KV ? pr->mem_cap * d_lane - pr->mem_prompt * (double)P
                                                                : (pr->mem_cap - pr->mem_prompt * (double)P / d) * d_lane;
          if (room < 0) { n_cand += (int)std::min<int64_t>(b_max, cdiv64(G, s)); continue; }
          cap = (int64_t)std::floor(room / pr->mem_resp);
          if (cap < 1) { n_cand += (int)std::min<int64_t>(b_max, cdiv64(G, s)); continue; }   // not even one token fits
        }
        // Up to the exact solver's limit one dynamic program per (primitive, s) serves every round count: its table
        // round_best[b][all units] is the optimum of Eq. 6 with at most b rounds.  Above the limit the greedy runs per b.
        const int b_hi = (int)std::min<int64_t>(b_max, cdiv64(G, s));
        const int exact_cap = std::min(t->exact_max_units > 0 ? t->exact_max_units : 12, kHardMaxExact);
        const bool use_dp = G <= exact_cap;
        // the program depends on (s, cell limit) alone: shared by degrees and primitives that agree on both
        ExactGrid *dp_ptr = nullptr;
        if (use_dp) {
          auto key = std::make_pair(s, cap);
          auto it = dp_cache.find(key);
          if (it == dp_cache.end()) {
            it = dp_cache.emplace(key, ExactGrid()).first;
            it->second.U = G; it->second.b = (int)std::min<int64_t>(b_max, G); it->second.s = std::min(s, G);
            it->second.solve(w.data(), m.data(), cap);
          }
          dp_ptr = &it->second;
        }
        for (int b = 1; b <= b_hi; ++b) {
          ++n_cand;
          int64_t work = 0;
          int32_t exact = 0;
          if (use_dp) {
            work = dp_ptr->round_best[b][(1u << G) - 1];
            if (work >= kInf) continue;  // the units do not fit this grid
            exact = 1;
          } else {
            const int r = assign_grid_impl(w.data(), m.data(), G, b, s, cap, t->exact_max_units, rounds.data(), lanes.data(), &work, &exact);
            if (r == AUGTREE_ERR_UNSUPPORTED) continue;
            if (r) return r;
          }
          const double L = (double)(cdiv64(G, (int64_t)b * s) * r_max);
          double replay, gamma;
          int d_eff;
          if (primitive == AUGTREE_TREE_MOVE_KV) {
            d_eff = d_lane;
            const double c_kv = b * 2 * ((double)P + L) * t->h_kv * f_ring(d_lane);
            replay = pr->alpha_tmkv * (double)work / d_lane + pr->beta_tmkv * c_kv + pr->lat_tmkv0 + pr->lat_tmkv1 * b * d_lane;
            gamma = pr->gamma_tmkv;
          } else {
            d_eff = d;
            const double c_q = b * L * t->h_q;
            const double t_r = b * (pr->red0 + pr->red1 * L * t->h_q) * f_ring(d);
            replay = pr->alpha_mq * (double)work / d_lane + pr->beta_q * c_q + t_r + pr->lat_mq0 + pr->lat_mq1 * b;
            gamma = pr->gamma_mq;
          }
          const double prefill = pr->alpha_p * (double)P / d_eff + pr->beta_p * (double)P * f_ring(d_eff) + pr->lat_p0 + pr->lat_p1 * d_eff;
          const double cost = gamma * (prefill + replay);
          if (!have || cost < best.cost) {
            have = true;
            best.cost = cost; best.degree = d; best.primitive = primitive; best.rounds = b; best.lanes = s; best.solved_exactly = exact;
            if (use_dp) dp_ptr->unpack(rounds.data(), lanes.data(), b);
            best_rounds = rounds; best_lanes = lanes;
          }
        }
      }
  }
  if (!have) return AUGTREE_ERR_UNSUPPORTED;
  best.n_candidates = n_cand;
  *choice = best;
  for (int k = 0; k < G; ++k) {
    round_out[k] = best.primitive == AUGTREE_RING_CP ? 0 : best_rounds[k];
    lane_out[k] = best.primitive == AUGTREE_RING_CP ? 0 : best_lanes[k];
  }
  return AUGTREE_OK;
}

extern "C" int augtree_plan_tree(const augtree_tree_t *tree, const augtree_profile_t *profile, augtree_choice_t *choice,
                                 int32_t *round_out, int32_t *lane_out) {
  try {
    return plan_tree_impl(tree, profile, choice, round_out, lane_out);
  } catch (...) {
    return AUGTREE_ERR_INTERNAL;
  }
}
