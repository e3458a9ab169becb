// Pack & schedule (host): prefix sums, work items for the six schedules (forward, key-side and query-side backward; prefill and replay call) and their
// largest-first assignment to replay lanes.
//
// Units and weights follow Sec. 3.4 ("Replay units and grid assignment"): a
// unit's weight is its valid Q-KV tile count, and units are placed on lanes so
// that the heaviest lane is as light as possible (Eq. 6 with one round), by
// largest-first greedy balancing.  On one GPU a lane is a persistent CTA, so a
// unit is one (query tile, head) for the forward kernels and one (KV tile, KV
// head) for the backward kernels rather than a whole response path.
//
// Canonical item order (ids are positions in this order):
//   prefill fwd : group, kv head, query tile, query head inside the kv head
//   replay  fwd : group, kv head, branch, query tile, query head, prompt-KV shard
//   replay  bwd : group, kv head, [prompt kv tiles, then branch by branch its kv tiles]   (dK, dV)
//   prefill bwd : group, kv head, kv tile                                                 (dK, dV)
//   replay  dQ  : group, kv head, branch, query tile, query head   (never sharded)
//   prefill dQ  : as prefill fwd
// Assignment: ids sorted by (weight descending, id ascending); each goes to the
// lane with the smallest load so far (lowest lane index on ties).  Inside a
// lane items run in ascending id, which keeps lanes on the same kv head at
// about the same time so that the head's K/V stay in L2.
#include "plan.h"

#include <algorithm>
#include <cmath>
#include <numeric>
#include <queue>

namespace augtree {

static inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// Returns false when the sizes do not fit the packed heap keys (lane index in 20 bits, lane load above them).
static bool assign_lanes(Sched &s, int weight_field, int n_lanes) {
  const int n = s.n_items();
  const int32_t *it = s.items.data();
  const int ni = s.item_ints;
  // ids by weight descending, id ascending inside a weight: a counting sort (weights are tile counts, small integers)
  int32_t wmax = 0;
  int64_t wsum = 0;
  for (int i = 0; i < n; ++i) { wmax = std::max(wmax, it[(size_t)i * ni + weight_field]); wsum += it[(size_t)i * ni + weight_field]; }
  if (n_lanes > (1 << 20) || wsum >= ((int64_t)1 << 43)) return false;
  std::vector<int32_t> ids(n);
  if ((int64_t)wmax <= 4 * (int64_t)n + 1024) {
    std::vector<int32_t> start((size_t)wmax + 2, 0);
    for (int i = 0; i < n; ++i) ++start[(size_t)(wmax - it[(size_t)i * ni + weight_field]) + 1];
    for (size_t b = 1; b < start.size(); ++b) start[b] += start[b - 1];
    for (int i = 0; i < n; ++i) ids[start[(size_t)(wmax - it[(size_t)i * ni + weight_field])]++] = i;
  } else {
    std::iota(ids.begin(), ids.end(), 0);
    std::stable_sort(ids.begin(), ids.end(), [&](int32_t a, int32_t b) {
      return it[(size_t)a * ni + weight_field] > it[(size_t)b * ni + weight_field];
    });
  }
  // largest first, each to the lane with the smallest (load, lane index): a binary min-heap of keys
  // load * 2^20 + lane whose top is replaced in place (one sift-down per item)
  std::vector<uint64_t> heap(n_lanes);
  std::vector<int32_t> lane_of(n), count(n_lanes + 1, 0);
  for (int l = 0; l < n_lanes; ++l) heap[l] = (uint64_t)l;   // all loads 0: ascending lane index is a valid heap
  uint64_t *hp = heap.data();
  for (int32_t id : ids) {
    const int32_t lane = (int32_t)(hp[0] & 0xfffffu);
    lane_of[id] = lane;
    ++count[lane + 1];
    const uint64_t key = hp[0] + ((uint64_t)it[(size_t)id * ni + weight_field] << 20);
    int i = 0;
    while (true) {
      int c = 2 * i + 1;
      if (c >= n_lanes) break;
      if (c + 1 < n_lanes && hp[c + 1] < hp[c]) ++c;
      if (hp[c] >= key) break;
      hp[i] = hp[c];
      i = c;
    }
    hp[i] = key;
  }
  // inside a lane items run in ascending id: one pass over the ids in order
  s.lane_ptr.assign(n_lanes + 1, 0);
  for (int l = 0; l < n_lanes; ++l) s.lane_ptr[l + 1] = s.lane_ptr[l] + count[l + 1];
  s.order.assign(n, 0);
  std::vector<int32_t> fill(s.lane_ptr.begin(), s.lane_ptr.end() - 1);
  for (int i = 0; i < n; ++i) s.order[fill[lane_of[i]]++] = i;
  return true;
}

int build_plan_host(const augtree_desc_t *d, augtree_plan *p) {
  if (!d || !p) return AUGTREE_ERR_INVALID_ARG;
  if (d->struct_size != sizeof(augtree_desc_t) || d->version != AUGTREE_VERSION) return AUGTREE_ERR_INVALID_ARG;
  if (d->n_groups < 1 || !d->prompt_len || !d->n_branches) return AUGTREE_ERR_INVALID_ARG;
  if (d->h_q < 1 || d->h_kv < 1 || d->n_lanes < 0 || d->kv_splits < 0) return AUGTREE_ERR_INVALID_ARG;
  if (d->h_q % d->h_kv != 0) return AUGTREE_ERR_UNSUPPORTED;
  // tiles are 64 or 128 columns wide; a head dimension below that is padded with zero columns by the tensor maps
  if (d->head_dim < 8 || d->head_dim > 128 || d->head_dim % 8 != 0) return AUGTREE_ERR_UNSUPPORTED;
  if (!(d->softmax_scale >= 0.f) || std::isinf(d->softmax_scale)) return AUGTREE_ERR_INVALID_ARG;

  p->n_groups = d->n_groups;
  p->h_q = d->h_q; p->h_kv = d->h_kv; p->head_dim = d->head_dim;
  p->scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / std::sqrt((float)d->head_dim);
  p->flags = d->flags;
  p->n_lanes = d->n_lanes;
  p->kv_splits = d->kv_splits < 1 ? 1 : d->kv_splits;
  if (p->kv_splits > 64 || p->h_kv > 64) return AUGTREE_ERR_UNSUPPORTED;

  p->prompt_len.assign(d->prompt_len, d->prompt_len + d->n_groups);
  p->n_br.assign(d->n_branches, d->n_branches + d->n_groups);
  int64_t nb = 0, tp = 0;
  p->cu_p.assign(1, 0); p->cu_b.assign(1, 0);
  for (int g = 0; g < d->n_groups; ++g) {
    if (p->prompt_len[g] < 1 || p->n_br[g] < 0) return AUGTREE_ERR_INVALID_ARG;
    tp += p->prompt_len[g]; nb += p->n_br[g];
    if (tp > 0x3fffffff || nb > 0x3fffffff) return AUGTREE_ERR_UNSUPPORTED;
    p->cu_p.push_back((int32_t)tp); p->cu_b.push_back((int32_t)nb);
  }
  if (nb > 0 && !d->branch_len) return AUGTREE_ERR_INVALID_ARG;
  p->n_branches = (int32_t)nb;
  p->branch_len.assign(d->branch_len, d->branch_len + nb);
  int64_t tr = 0;
  p->cu_r.assign(1, 0);
  for (int64_t i = 0; i < nb; ++i) {
    if (p->branch_len[i] < 1) return AUGTREE_ERR_INVALID_ARG;
    tr += p->branch_len[i];
    if (tr > 0x3fffffff) return AUGTREE_ERR_UNSUPPORTED;
    p->cu_r.push_back((int32_t)tr);
  }
  p->total_p = tp; p->total_r = tr;
  p->branch_group.resize(nb);
  for (int g = 0; g < d->n_groups; ++g)
    for (int i = p->cu_b[g]; i < p->cu_b[g + 1]; ++i) p->branch_group[i] = g;

  const int rep = p->h_q / p->h_kv;
  const int ng = p->n_groups;

  // q-segment tables for the backward kernels
  // (a segment's 128-row query tiles are numbered consecutively; the per-row
  // statistics of the backward pass are stored tile by tile in that numbering)
  p->seg_replay.clear(); p->seg_prefill.clear(); p->tiles_replay.clear(); p->tiles_prefill.clear();
  auto add_segment = [](std::vector<int32_t> &segs, std::vector<int32_t> &tiles, int tok0, int len) {
    segs.push_back(tok0); segs.push_back(len); segs.push_back((int32_t)(tiles.size() / 2));
    for (int t = 0; t < cdiv(len, kTileQ); ++t) { tiles.push_back(tok0 + t * kTileQ); tiles.push_back(std::min(kTileQ, len - t * kTileQ)); }
  };
  for (int i = 0; i < (int)nb; ++i) add_segment(p->seg_replay, p->tiles_replay, p->cu_r[i], p->branch_len[i]);
  for (int g = 0; g < ng; ++g) add_segment(p->seg_prefill, p->tiles_prefill, p->cu_p[g], p->prompt_len[g]);

  // dS hand-off tables: query tile t of a backward call sees n_t KV tiles (the group's prompt tiles in the replay call,
  // then the causal tiles of its own sequence); its (head, KV tile) pairs own consecutive 128 x 128 slots of the scratch
  p->pairs_replay.clear(); p->pairs_prefill.clear();
  auto add_pairs = [](std::vector<int32_t> &tab, int64_t &slots, int len, int n_prompt_tiles) {
    for (int t = 0; t < cdiv(len, kTileQ); ++t) {
      const int n = n_prompt_tiles + t + 1;
      const int32_t e[4] = {(int32_t)slots, n, n_prompt_tiles, 0};
      tab.insert(tab.end(), e, e + 4);
      slots += n;
    }
  };
  p->ds_slots_replay = p->ds_slots_prefill = 0;
  for (int i = 0; i < (int)nb; ++i)
    add_pairs(p->pairs_replay, p->ds_slots_replay, p->branch_len[i], cdiv(p->prompt_len[p->branch_group[i]], kTileKV));
  for (int g = 0; g < ng; ++g) add_pairs(p->pairs_prefill, p->ds_slots_prefill, p->prompt_len[g], 0);

  // prompt-KV shards per group: shard = a run of whole KV tiles
  p->group_splits.resize(ng);
  std::vector<int> shard_tiles(ng);
  p->max_splits = 1;
  for (int g = 0; g < ng; ++g) {
    const int na = cdiv(p->prompt_len[g], kTileKV);
    const int want = std::min(p->kv_splits, na);
    shard_tiles[g] = cdiv(na, want);
    p->group_splits[g] = cdiv(na, shard_tiles[g]);
    p->max_splits = std::max(p->max_splits, p->group_splits[g]);
  }

  Sched &pf = p->sched[SCHED_PREFILL_FWD], &rf = p->sched[SCHED_REPLAY_FWD];
  Sched &rb = p->sched[SCHED_REPLAY_BWD], &pb = p->sched[SCHED_PREFILL_BWD];
  Sched &rq = p->sched[SCHED_REPLAY_DQ], &pq = p->sched[SCHED_PREFILL_DQ];
  pf.item_ints = rf.item_ints = rq.item_ints = pq.item_ints = AUGTREE_FWD_ITEM_INTS;
  rb.item_ints = pb.item_ints = AUGTREE_BWD_ITEM_INTS;
  pf.items.clear(); rf.items.clear(); rb.items.clear(); pb.items.clear(); rq.items.clear(); pq.items.clear();
  {  // item counts, so that the tables below grow without reallocation
    size_t n_pf = 0, n_rf = 0, n_rb = 0, n_pb = 0, n_rq = 0, n_pq = 0;
    for (int g = 0; g < ng; ++g) {
      const int P = p->prompt_len[g];
      n_pf += (size_t)cdiv(P, kTileQF) * p->h_q;
      n_pq += (size_t)cdiv(P, kTileQ) * p->h_q;
      n_pb += (size_t)cdiv(P, kTileKV) * p->h_kv;
      if (p->cu_b[g + 1] > p->cu_b[g]) n_rb += (size_t)cdiv(P, kTileKV) * p->h_kv;
      for (int b = p->cu_b[g]; b < p->cu_b[g + 1]; ++b) {
        const int R = p->branch_len[b];
        n_rq += (size_t)cdiv(R, kTileQ) * p->h_q;
        n_rf += (size_t)cdiv(R, kTileQF) * p->h_q * p->group_splits[g];
        n_rb += (size_t)cdiv(R, kTileKV) * p->h_kv;
      }
    }
    pf.items.reserve(n_pf * AUGTREE_FWD_ITEM_INTS); rf.items.reserve(n_rf * AUGTREE_FWD_ITEM_INTS);
    rq.items.reserve(n_rq * AUGTREE_FWD_ITEM_INTS); pq.items.reserve(n_pq * AUGTREE_FWD_ITEM_INTS);
    rb.items.reserve(n_rb * AUGTREE_BWD_ITEM_INTS); pb.items.reserve(n_pb * AUGTREE_BWD_ITEM_INTS);
  }

  for (int g = 0; g < ng; ++g) {
    const int P = p->prompt_len[g], p0 = p->cu_p[g];
    const int nqt_p = cdiv(P, kTileQ);
    for (int c = 0; c < p->h_kv; ++c) {
      // ---- prefill forward: units of two query tiles (256 rows) ----
      for (int t = 0; t < cdiv(P, kTileQF); ++t) {
        const int rows = std::min(kTileQF, P - t * kTileQF);
        const int blen = t * kTileQF + rows;
        for (int j = 0; j < rep; ++j) {
          const int32_t it[AUGTREE_FWD_ITEM_INTS] = {p0 + t * kTileQF, t * kTileQF, rows, c * rep + j, 0, 0, p0, blen,
                                                     0, 1, cdiv(blen, kTileKV) * cdiv(rows, kTileQ), c};
          pf.items.insert(pf.items.end(), it, it + AUGTREE_FWD_ITEM_INTS);
        }
      }
      // ---- prefill dQ: units of one query tile; field 8 is the tile's index in the per-tile row statistics ----
      for (int t = 0; t < nqt_p; ++t) {
        const int rows = std::min(kTileQ, P - t * kTileQ);
        const int blen = t * kTileQ + rows;
        for (int j = 0; j < rep; ++j) {
          const int32_t dq[AUGTREE_FWD_ITEM_INTS] = {p0 + t * kTileQ, t * kTileQ, rows, c * rep + j, 0, 0, p0, blen,
                                                     p->seg_prefill[3 * g + 2] + t, 1, cdiv(blen, kTileKV), c};
          pq.items.insert(pq.items.end(), dq, dq + AUGTREE_FWD_ITEM_INTS);
        }
      }
      // ---- replay forward (256-row units, optionally sharded over the prompt KV) and replay dQ (128-row units) ----
      for (int b = p->cu_b[g]; b < p->cu_b[g + 1]; ++b) {
        const int R = p->branch_len[b], r0 = p->cu_r[b];
        const int ns = p->group_splits[g];
        for (int t = 0; t < cdiv(R, kTileQ); ++t) {
          const int rows = std::min(kTileQ, R - t * kTileQ);
          const int blen = t * kTileQ + rows;
          for (int j = 0; j < rep; ++j) {
            const int32_t dq[AUGTREE_FWD_ITEM_INTS] = {r0 + t * kTileQ, t * kTileQ, rows, c * rep + j, p0, P, r0, blen,
                                                       p->seg_replay[3 * b + 2] + t, 1, cdiv(P, kTileKV) + cdiv(blen, kTileKV), c};
            rq.items.insert(rq.items.end(), dq, dq + AUGTREE_FWD_ITEM_INTS);
          }
        }
        for (int t = 0; t < cdiv(R, kTileQF); ++t) {
          const int rows = std::min(kTileQF, R - t * kTileQF);
          const int blen = t * kTileQF + rows;
          for (int j = 0; j < rep; ++j)
            for (int s = 0; s < ns; ++s) {
              const int a0 = s * shard_tiles[g] * kTileKV;
              const int alen = std::min(P - a0, shard_tiles[g] * kTileKV);
              const int bl = (s == ns - 1) ? blen : 0;
              const int32_t it[AUGTREE_FWD_ITEM_INTS] = {r0 + t * kTileQF, t * kTileQF, rows, c * rep + j, p0 + a0, alen,
                                                         r0, bl, s, ns, (cdiv(alen, kTileKV) + cdiv(bl, kTileKV)) * cdiv(rows, kTileQ), c};
              rf.items.insert(rf.items.end(), it, it + AUGTREE_FWD_ITEM_INTS);
            }
        }
      }
      // ---- replay backward: prompt kv tiles (mode 1), then each branch's kv tiles (mode 0) ----
      const int b0 = p->cu_b[g], b1 = p->cu_b[g + 1];
      if (b1 > b0) {
        int visits = 0;
        for (int b = b0; b < b1; ++b) visits += cdiv(p->branch_len[b], kTileQ) * rep;
        for (int t = 0; t < cdiv(P, kTileKV); ++t) {
          const int32_t it[AUGTREE_BWD_ITEM_INTS] = {p0 + t * kTileKV, t * kTileKV, std::min(kTileKV, P - t * kTileKV), c,
                                                     1, b0, b1 - b0, visits};
          rb.items.insert(rb.items.end(), it, it + AUGTREE_BWD_ITEM_INTS);
        }
      }
      for (int b = b0; b < b1; ++b) {
        const int R = p->branch_len[b], r0 = p->cu_r[b];
        const int nt = cdiv(R, kTileKV);
        for (int t = 0; t < nt; ++t) {
          const int32_t it[AUGTREE_BWD_ITEM_INTS] = {r0 + t * kTileKV, t * kTileKV, std::min(kTileKV, R - t * kTileKV), c,
                                                     0, b, 1, (cdiv(R, kTileQ) - t) * rep};
          rb.items.insert(rb.items.end(), it, it + AUGTREE_BWD_ITEM_INTS);
        }
      }
      // ---- prefill backward ----
      for (int t = 0; t < cdiv(P, kTileKV); ++t) {
        const int32_t it[AUGTREE_BWD_ITEM_INTS] = {p0 + t * kTileKV, t * kTileKV, std::min(kTileKV, P - t * kTileKV), c,
                                                   0, g, 1, (nqt_p - t) * rep};
        pb.items.insert(pb.items.end(), it, it + AUGTREE_BWD_ITEM_INTS);
      }
    }
  }
  if (p->n_lanes > 0) {
    if (!assign_lanes(pf, 10, p->n_lanes) || !assign_lanes(rf, 10, p->n_lanes) || !assign_lanes(rb, 7, p->n_lanes) ||
        !assign_lanes(pb, 7, p->n_lanes) || !assign_lanes(rq, 10, p->n_lanes) || !assign_lanes(pq, 10, p->n_lanes))
      return AUGTREE_ERR_UNSUPPORTED;
  }

  // scratch sizes (bytes, each region 256-byte aligned)
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  const size_t hq = (size_t)p->h_q, dd = (size_t)p->head_dim;
  // forward: 256 bytes for the per-KV-head key-norm maxima, then (with prompt-KV shards) the shards' partial states
  p->ws_fwd = 256;
  if (p->max_splits > 1)
    p->ws_fwd += al((size_t)p->max_splits * (size_t)tr * hq * dd * 4) + al((size_t)p->max_splits * (size_t)tr * hq * 4);
  const size_t tmax = (size_t)std::max<int64_t>(tp, tr);
  // backward: row statistics [H_q][tiles][2][128] fp32
  const size_t ntile = std::max(p->tiles_replay.size(), p->tiles_prefill.size()) / 2;
  p->ws_bwd = al(hq * ntile * 2 * kTileQ * 4);
  // with this much, the key-side kernel also stores dS (bf16, one 128 x 128 tile per pair and head) for the query side
  const int64_t ds_slots = std::max(p->ds_slots_replay, p->ds_slots_prefill);
  // (slot indices are 32-bit tensor-map coordinates)
  p->ws_bwd_handoff = ds_slots * (int64_t)p->h_q > 0x7fffffff ? ~(size_t)0 : p->ws_bwd + al((size_t)ds_slots * hq * (size_t)(kTileQ * kTileKV * 2));
  (void)tmax; (void)dd;
  return AUGTREE_OK;
}

}  // namespace augtree
