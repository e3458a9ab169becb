"""Independent restatement of the pack-and-schedule metadata (test infrastructure only).

Written from the rules, not from the library's source: the tests demand that
the library's tables equal these bit for bit.  What pins THESE tables is not
the library but tests/test_packing_cover.py: every item is expanded from its
fields into the (query, key, head) triples it stands for, and each schedule
must cover the tree mask of Eq. 1 exactly once, with weights equal to visited
tile counts and one owner per prompt-KV tile.

Rules.  Tiles are 128 query rows by 128 keys.  A forward item is one (pair of
consecutive query tiles, query head[, prompt-KV shard]); its weight is the
number of (query tile, KV tile) visits.  A dQ item is one (query tile, query
head), weighted by its KV tiles.  A backward item is one (KV tile, KV head); its weight is the number of
(query tile, query head) visits.  Items are listed in a canonical order, then
assigned to lanes largest weight first (ties: lower id first), each to the lane
with the least load so far (ties: lowest lane), following the balanced
makespan assignment of Sec. 3.4 / Eq. 6 in its greedy form; a lane runs its
items in ascending id.
"""
from __future__ import annotations

import heapq

import numpy as np

TQ = TK = 128
TQF = 256   # forward units cover two query tiles


def _cdiv(a, b):
    return -(-a // b)


def prefix(xs):
    out = [0]
    for x in xs:
        out.append(out[-1] + x)
    return out


def build_tables(prompt_len, branch_len, h_q, h_kv, kv_splits=1):
    rep = h_q // h_kv
    cu_p = prefix(prompt_len)
    cu_b = prefix([len(b) for b in branch_len])
    flat = [r for b in branch_len for r in b]
    cu_r = prefix(flat)
    kv_splits = max(1, kv_splits)
    pf, rf, rb, pb, gsplits, rq, pq = [], [], [], [], [], [], []
    ptile0 = prefix([_cdiv(x, TQ) for x in prompt_len])
    rtile0 = prefix([_cdiv(x, TQ) for x in flat])
    for g, P in enumerate(prompt_len):
        p0 = cu_p[g]
        na = _cdiv(P, TK)
        shard_tiles = _cdiv(na, min(kv_splits, na))
        ns = _cdiv(na, shard_tiles)
        gsplits.append(ns)
        for c in range(h_kv):
            for t in range(_cdiv(P, TQF)):      # forward units: two query tiles
                rows = min(TQF, P - t * TQF)
                vis = t * TQF + rows
                for j in range(rep):
                    pf.append([p0 + t * TQF, t * TQF, rows, c * rep + j, 0, 0, p0, vis, 0, 1, _cdiv(vis, TK) * _cdiv(rows, TQ), c])
            for t in range(_cdiv(P, TQ)):       # dQ units: one query tile
                rows = min(TQ, P - t * TQ)
                vis = t * TQ + rows
                for j in range(rep):
                    pq.append([p0 + t * TQ, t * TQ, rows, c * rep + j, 0, 0, p0, vis, ptile0[g] + t, 1, _cdiv(vis, TK), c])
            for bi in range(cu_b[g], cu_b[g + 1]):
                R, r0 = flat[bi], cu_r[bi]
                for t in range(_cdiv(R, TQ)):
                    rows = min(TQ, R - t * TQ)
                    vis = t * TQ + rows
                    for j in range(rep):
                        rq.append([r0 + t * TQ, t * TQ, rows, c * rep + j, p0, P, r0, vis, rtile0[bi] + t, 1,
                                   _cdiv(P, TK) + _cdiv(vis, TK), c])
                for t in range(_cdiv(R, TQF)):
                    rows = min(TQF, R - t * TQF)
                    vis = t * TQF + rows
                    for j in range(rep):
                        for s in range(ns):
                            a0 = s * shard_tiles * TK
                            alen = min(P - a0, shard_tiles * TK)
                            bl = vis if s == ns - 1 else 0
                            rf.append([r0 + t * TQF, t * TQF, rows, c * rep + j, p0 + a0, alen, r0, bl, s, ns,
                                       (_cdiv(alen, TK) + _cdiv(bl, TK)) * _cdiv(rows, TQ), c])
            b0, b1 = cu_b[g], cu_b[g + 1]
            if b1 > b0:
                visits = sum(_cdiv(flat[bi], TQ) * rep for bi in range(b0, b1))
                for t in range(_cdiv(P, TK)):
                    rb.append([p0 + t * TK, t * TK, min(TK, P - t * TK), c, 1, b0, b1 - b0, visits])
            for bi in range(b0, b1):
                R, r0 = flat[bi], cu_r[bi]
                for t in range(_cdiv(R, TK)):
                    rb.append([r0 + t * TK, t * TK, min(TK, R - t * TK), c, 0, bi, 1, (_cdiv(R, TQ) - t) * rep])
            for t in range(_cdiv(P, TK)):
                pb.append([p0 + t * TK, t * TK, min(TK, P - t * TK), c, 0, g, 1, (_cdiv(P, TQ) - t) * rep])
    arr = lambda x, w: np.asarray(x, dtype=np.int32).reshape(-1, w)
    return {
        "cu_p": np.asarray(cu_p, np.int32), "cu_b": np.asarray(cu_b, np.int32), "cu_r": np.asarray(cu_r, np.int32),
        "prefill_fwd": arr(pf, 12), "replay_fwd": arr(rf, 12), "replay_bwd": arr(rb, 8), "prefill_bwd": arr(pb, 8),
        "replay_dq": arr(rq, 12), "prefill_dq": arr(pq, 12),
        "group_splits": np.asarray(gsplits, np.int32),
        # segments: first token, length, index of the segment's first 128-row query tile
        "seg_replay": np.asarray([[cu_r[i], flat[i], sum(_cdiv(x, TQ) for x in flat[:i])] for i in range(len(flat))],
                                 np.int32).reshape(-1, 3),
        "seg_prefill": np.asarray([[cu_p[g], prompt_len[g], sum(_cdiv(x, TQ) for x in prompt_len[:g])]
                                   for g in range(len(prompt_len))], np.int32).reshape(-1, 3),
    }


def assign_lanes(weights, n_lanes):
    """Largest-first greedy assignment.  Returns (lane_ptr [n_lanes+1], order [n])."""
    ids = sorted(range(len(weights)), key=lambda i: (-int(weights[i]), i))
    heap = [(0, l) for l in range(n_lanes)]
    heapq.heapify(heap)
    lanes = [[] for _ in range(n_lanes)]
    for i in ids:
        load, l = heapq.heappop(heap)
        lanes[l].append(i)
        heapq.heappush(heap, (load + int(weights[i]), l))
    order, ptr = [], [0]
    for l in range(n_lanes):
        order += sorted(lanes[l])
        ptr.append(len(order))
    return np.asarray(ptr, np.int32), np.asarray(order, np.int32)


def makespan(weights, lane_ptr, order):
    w = np.asarray(weights)
    return max(int(w[order[lane_ptr[l]:lane_ptr[l + 1]]].sum()) for l in range(len(lane_ptr) - 1))


def brute_force_makespan(weights, n_lanes):
    """Optimal makespan by exhaustive assignment (tiny inputs only)."""
    best = [sum(weights)]
    loads = [0] * n_lanes

    def rec(i):
        if i == len(weights):
            best[0] = min(best[0], max(loads))
            return
        seen = set()
        for l in range(n_lanes):
            if loads[l] in seen:
                continue
            seen.add(loads[l])
            loads[l] += weights[i]
            if max(loads) < best[0]:
                rec(i + 1)
            loads[l] -= weights[i]
    rec(0)
    return best[0]


# --------------------------------------------------------------------------- #
# Replay-grid assignment (Sec. 3.4 "Replay units and grid assignment", Eq. 6).
#
# Units k = 0..U-1 with work w_k are placed on a grid of b rounds x s lanes,
# X_k = (round, lane).  Lanes of a round run concurrently and rounds run one
# after the other, so the predicted critical path is
#     sum over rounds of ( max over lanes of ( sum of w_k placed there ) ).
# The paper adds per-lane memory limits; here a unit also has a size m_k and a
# (round, lane) cell holds at most `cap` of it (cap None: no limit).  Without a
# limit one round is always enough, because merging rounds never lengthens the
# path; the limit is what makes several rounds necessary.
#
# grid_objective is Eq. 6 written out; brute_force_grid is its definition as a
# minimum over every assignment (tiny inputs only); greedy_grid restates the
# largest-first rule the library uses above the exact-solver cap, tie-breaks
# included, for a bit-exact comparison.  Test infrastructure only.


def grid_objective(weights, rounds, lanes, n_rounds, n_lanes):
    load = np.zeros((n_rounds, n_lanes), dtype=np.int64)
    for w, t, j in zip(weights, rounds, lanes):
        load[t, j] += int(w)
    return int(load.max(axis=1).sum())


def grid_feasible(mem, rounds, lanes, n_rounds, n_lanes, cap):
    if cap is None:
        return True
    used = np.zeros((n_rounds, n_lanes), dtype=np.int64)
    for m, t, j in zip(mem, rounds, lanes):
        used[t, j] += int(m)
    return bool((used <= cap).all())


def brute_force_grid(weights, mem, n_rounds, n_lanes, cap):
    """Minimum of Eq. 6 over all (n_rounds * n_lanes)^U assignments; None if no assignment fits the limit."""
    import itertools
    cells = [(t, j) for t in range(n_rounds) for j in range(n_lanes)]
    best = None
    for choice in itertools.product(range(len(cells)), repeat=len(weights)):
        rounds = [cells[c][0] for c in choice]
        lanes = [cells[c][1] for c in choice]
        if not grid_feasible(mem, rounds, lanes, n_rounds, n_lanes, cap):
            continue
        v = grid_objective(weights, rounds, lanes, n_rounds, n_lanes)
        if best is None or v < best:
            best = v
    return best


def greedy_grid(weights, mem, n_rounds, n_lanes, cap):
    """Largest-first greedy: units by weight descending (index ascending on ties); each goes to the cell that
    fits and gives the smallest critical path afterwards, then the smallest cell load, then the lowest round,
    then the lowest lane.  Returns (rounds, lanes, objective) or None if some unit fits nowhere."""
    U = len(weights)
    load = [[0] * n_lanes for _ in range(n_rounds)]
    used = [[0] * n_lanes for _ in range(n_rounds)]
    rounds, lanes = [0] * U, [0] * U
    for k in sorted(range(U), key=lambda i: (-int(weights[i]), i)):
        best = None
        for t in range(n_rounds):
            peak = max(load[t])
            for j in range(n_lanes):
                if cap is not None and used[t][j] + int(mem[k]) > cap:
                    continue
                new = load[t][j] + int(weights[k])
                key = (max(peak, new) - peak, new, t, j)  # growth of this round's maximum = growth of the path
                if best is None or key < best[0]:
                    best = (key, t, j)
        if best is None:
            return None
        _, t, j = best
        load[t][j] += int(weights[k])
        used[t][j] += int(mem[k])
        rounds[k], lanes[k] = t, j
    return rounds, lanes, sum(max(r) for r in load)
