// Internal plan object: packing metadata on the host and its device copies.
#pragma once
#include <atomic>
#include <cstdint>
#include <vector>

#include "../../include/augtree.h"

namespace augtree {

constexpr int kTileQ = 128;   // query rows per tile
constexpr int kTileQF = 256;  // query rows per forward unit (two tiles share every K/V tile they load)
constexpr int kTileKV = 128;  // keys per tile

enum { SCHED_PREFILL_FWD = 0, SCHED_REPLAY_FWD = 1, SCHED_REPLAY_BWD = 2, SCHED_PREFILL_BWD = 3, SCHED_REPLAY_DQ = 4, SCHED_PREFILL_DQ = 5,
       SCHED_COUNT = 6 };

constexpr int kStatusInts = 2 + SCHED_COUNT;

struct Sched {
  int item_ints = 0;
  std::vector<int32_t> items;     // canonical order, item_ints per item
  std::vector<int32_t> lane_ptr;  // [n_lanes + 1]
  std::vector<int32_t> order;     // item ids, lane by lane
  int32_t *d_items = nullptr;     // items gathered into lane order (device)
  int32_t *d_lane_ptr = nullptr;  // (device)
  int n_items() const { return item_ints ? (int)(items.size() / item_ints) : 0; }
};

// CUDA-event pairs recorded around the tile kernels when timing is switched on.
struct Timing {
  bool on = false;
  std::vector<void *> ev[SCHED_COUNT];  // cudaEvent_t start/stop pairs, in launch order
  size_t used[SCHED_COUNT] = {};
};

}  // namespace augtree

struct augtree_plan {
  int32_t n_groups = 0, n_branches = 0;
  int32_t h_q = 0, h_kv = 0, head_dim = 0;
  float scale = 0.f;
  uint32_t flags = 0;
  int32_t n_lanes = 0, kv_splits = 1, max_splits = 1;
  int device = -1;
  int64_t total_p = 0, total_r = 0;
  std::vector<int32_t> prompt_len, n_br, branch_len;
  std::vector<int32_t> cu_p, cu_b, cu_r, branch_group, group_splits;
  std::vector<int32_t> seg_replay, seg_prefill;    // [n][3] {first query token, length, first tile index}
  std::vector<int32_t> tiles_replay, tiles_prefill;  // [n_tiles][2] {first token, rows}: 128-row query tiles per segment
  // dS hand-off of the backward pass: per query tile {first slot / heads, KV tiles it sees, prompt KV tiles among them, 0}
  std::vector<int32_t> pairs_replay, pairs_prefill;
  int64_t ds_slots_replay = 0, ds_slots_prefill = 0;  // (KV tile, query tile) pairs per head of each backward call
  augtree::Sched sched[augtree::SCHED_COUNT];
  int32_t *d_seg_replay = nullptr, *d_seg_prefill = nullptr, *d_branch_group = nullptr, *d_group_splits = nullptr;
  int32_t *d_cu_r = nullptr;
  int32_t *d_tiles_replay = nullptr, *d_tiles_prefill = nullptr;
  int32_t *d_pairs_replay = nullptr, *d_pairs_prefill = nullptr;
  int *d_status = nullptr;  // [kStatusInts]: status, detail, then the items each schedule's kernel has finished
  mutable std::atomic<long long> launched_items[augtree::SCHED_COUNT] = {};  // items handed to launches so far
  augtree::Timing *timing = nullptr;  // optional CUDA-event timing of the tile kernels
  size_t ws_fwd = 0, ws_bwd = 0;
  size_t ws_bwd_handoff = 0;  // backward scratch at which the key-side kernel hands dS to the query-side kernel
};

namespace augtree {
int build_plan_host(const augtree_desc_t *desc, augtree_plan *plan);
}
