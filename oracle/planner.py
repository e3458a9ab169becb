"""Oracle of the online strategy planner (Sec. 3.4, Algorithm 1, Eq. 6-10).  TEST INFRASTRUCTURE ONLY.

Plain restatement: enumerate every candidate c = (d, pi, (b, s), X), place the replay units with the
brute-force minimum of Eq. 6 (oracle.packing.brute_force_grid: all assignments, tiny inputs only), score the
candidate with Eq. 7-10 and keep the cheapest.  Nothing here is shared with the library's planner.

The paper states the shape of the cost model and leaves its constants to profiling, so every constant is an
input (`Profile`).  Where the paper leaves a quantity's definition open, this file fixes a reading, marked
[reading] below; the library has to implement the same readings and the tests compare the two.

Notation as in the paper: L_P prompt length, R_i response lengths, G branches, d CP degree, s lanes per round,
b rounds, d_lane = d / s ranks per lane, X_k = (round, lane) of unit k, H_q / H_kv head counts.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

from oracle import packing

TILE = 128
RING_CP, TREE_MOVE_KV, MOVE_Q = 0, 1, 2     # primitive ids, also the enumeration order inside one degree


@dataclass
class Profile:
    """Constants of Eq. 7-10 (times in arbitrary but common units) and the memory model."""
    # Eq. 8, prompt prefill:  alpha_p L_P / d_eff + beta_p L_P f_ring(d_eff) + (lat_p0 + lat_p1 d_eff)
    alpha_p: float = 1.0
    beta_p: float = 0.0
    lat_p0: float = 0.0
    lat_p1: float = 0.0
    # Eq. 9, TreeMoveKV replay:  alpha W / d_lane + beta C_KV + (lat0 + lat1 b d_lane)
    alpha_tmkv: float = 1.0
    beta_tmkv: float = 0.0
    lat_tmkv0: float = 0.0
    lat_tmkv1: float = 0.0
    # Eq. 10, MoveQ replay:  alpha W / d_lane + beta_q C_Q + T_r + (lat0 + lat1 b)
    alpha_mq: float = 1.0
    beta_q: float = 0.0
    red0: float = 0.0          # T_r = sum over rounds of (red0 + red1 * reduced volume of the round) * f_ring(d)
    red1: float = 0.0
    lat_mq0: float = 0.0
    lat_mq1: float = 0.0
    # b = 0, ordinary ring CP over every (P, R_i) pair:  alpha tiles / d + beta 2 (L_P + R_i) H_kv f_ring(d) + (lat0 + lat1 d)
    alpha_ring: float = 1.0
    beta_ring: float = 0.0
    lat_ring0: float = 0.0
    lat_ring1: float = 0.0
    # Eq. 7 calibration factors gamma_c, one per primitive
    gamma_ring: float = 1.0
    gamma_tmkv: float = 1.0
    gamma_mq: float = 1.0
    # per-rank memory: capacity, bytes per resident prompt token, bytes per response token in flight (0 cap: no limit)
    mem_cap: float = 0.0
    mem_prompt: float = 0.0
    mem_resp: float = 1.0


def cdiv(a, b):
    return -(-a // b)


def f_ring(d):
    """[reading] fraction of a ring pass that crosses a link: (d - 1) / d (the paper leaves f_ring unspecified)."""
    return (d - 1) / d


def replay_tiles(P, R):
    """Valid Q-KV tiles of one response path in replay: every response query tile against every prompt tile, plus the
    causal triangle of its own tiles (the weight w_k of a replay unit in Sec. 3.4 is its count of valid tiles)."""
    nq = cdiv(R, TILE)
    return nq * cdiv(P, TILE) + nq * (nq + 1) // 2


def causal_tiles(n):
    nq = cdiv(n, TILE)
    return nq * (nq + 1) // 2


def divisors(d):
    return [s for s in range(1, d + 1) if d % s == 0]


def cell_token_cap(prof: Profile, primitive, P, d, s):
    """[reading] Largest number of response tokens one (round, lane) cell may hold.  TreeMoveKV: a lane of d_lane ranks
    holds the whole prompt state and its cell's tokens; MoveQ: the prompt state is spread over all d ranks and a cell's
    tokens over the d_lane ranks that serve the lane.  None: no limit; negative: the prompt alone does not fit."""
    if prof.mem_cap <= 0:
        return None
    d_lane = d // s
    if primitive == TREE_MOVE_KV:
        room = prof.mem_cap * d_lane - prof.mem_prompt * P
    else:
        room = (prof.mem_cap - prof.mem_prompt * P / d) * d_lane
    return int(room // prof.mem_resp) if room >= 0 else -1


def cell_tokens_proxy(R, b, s):
    """Response tokens of the fullest cell, estimated without looking at the placement: Sec. 3.4 lets the longest
    response length max_i |R_i| stand in, conservatively, for the replay length; here for ceil(G / (b s)) paths per cell
    [reading].  The traffic terms then depend on the candidate alone and the placement enters through W only."""
    return cdiv(len(R), b * s) * max(R)


def split_cost(prof: Profile, primitive, P, R, h_q, h_kv, d, b, s, work):
    """Eq. 7 for a split candidate (b >= 1) whose placement has critical-path work `work` (Eq. 6's objective)."""
    d_lane = d // s
    L = cell_tokens_proxy(R, b, s)
    if primitive == TREE_MOVE_KV:
        d_eff = d_lane                                                        # every lane prefills the prompt itself
        c_kv = b * 2 * (P + L) * h_kv * f_ring(d_lane)                        # Eq. 3, once per round
        replay = prof.alpha_tmkv * work / d_lane + prof.beta_tmkv * c_kv + prof.lat_tmkv0 + prof.lat_tmkv1 * b * d_lane
        gamma = prof.gamma_tmkv
    else:
        d_eff = d
        c_q = b * L * h_q                                                     # Eq. 4's query traffic, once per round
        t_r = b * (prof.red0 + prof.red1 * L * h_q) * f_ring(d)               # [reading] one reduction per round
        replay = prof.alpha_mq * work / d_lane + prof.beta_q * c_q + t_r + prof.lat_mq0 + prof.lat_mq1 * b
        gamma = prof.gamma_mq
    prefill = prof.alpha_p * P / d_eff + prof.beta_p * P * f_ring(d_eff) + prof.lat_p0 + prof.lat_p1 * d_eff   # Eq. 8
    return gamma * (prefill + replay)


def ring_cost(prof: Profile, P, R, h_q, h_kv, d):
    """b = 0: ordinary ring CP over every flattened pair (P, R_i), the prompt recomputed per branch."""
    total = 0.0
    for r in (R if R else [0]):
        total += prof.alpha_ring * causal_tiles(P + r) / d + prof.beta_ring * 2 * (P + r) * h_kv * f_ring(d) \
            + prof.lat_ring0 + prof.lat_ring1 * d
    return prof.gamma_ring * total


def ring_feasible(prof: Profile, P, R, d):
    if prof.mem_cap <= 0:
        return True
    longest = P + (max(R) if R else 0)
    return (prof.mem_prompt * P + prof.mem_resp * (longest - P)) / d <= prof.mem_cap


@dataclass
class Choice:
    cost: float
    d: int
    primitive: int
    b: int
    s: int
    rounds: List[int] = field(default_factory=list)
    lanes: List[int] = field(default_factory=list)


def candidates(P, R, degrees, b_max):
    """Algorithm 1's loops: degrees in the given order; per degree RingCP, then TreeMoveKV and MoveQ over lanes s | d with
    s <= G [reading: a lane count that leaves a lane without any unit is the same plan with fewer lanes] and rounds
    b = 1 .. min(b_max, ceil(G / s)) [reading: more rounds than one unit per cell needs are never useful]."""
    G = len(R)
    for d in degrees:
        yield d, RING_CP, 0, 1
        if G == 0:
            continue
        for primitive in (TREE_MOVE_KV, MOVE_Q):
            for s in divisors(d):
                if s > G:
                    continue
                for b in range(1, min(b_max, cdiv(G, s)) + 1):
                    yield d, primitive, b, s


def plan_tree(P, R, h_q, h_kv, degrees, prof: Profile, b_max=4) -> Optional[Choice]:
    """The cheapest feasible candidate (first in enumeration order on ties); None if nothing is feasible.
    Placement by exhaustive search over every assignment: for tiny G only."""
    best = None
    w = [replay_tiles(P, r) for r in R]
    for d, primitive, b, s in candidates(P, R, degrees, b_max):
        if primitive == RING_CP:
            if not ring_feasible(prof, P, R, d):
                continue
            cand = Choice(ring_cost(prof, P, R, h_q, h_kv, d), d, RING_CP, 0, 1)
        else:
            cap = cell_token_cap(prof, primitive, P, d, s)
            if cap is not None and cap < 0:
                continue
            placed = _best_placement(prof, primitive, P, R, w, h_q, h_kv, d, b, s, cap)
            if placed is None:
                continue
            cand = placed
        if best is None or cand.cost < best.cost:
            best = cand
    return best


def _best_placement(prof, primitive, P, R, w, h_q, h_kv, d, b, s, cap):
    """The AssignGrid step for one candidate: Eq. 6's minimum over all placements that respect the cell limit, by
    exhaustive search, and one placement that attains it."""
    import itertools
    target = packing.brute_force_grid(w, R, b, s, cap)
    if target is None:
        return None
    cost = split_cost(prof, primitive, P, R, h_q, h_kv, d, b, s, target)
    cells = [(t, j) for t in range(b) for j in range(s)]
    for choice in itertools.product(range(len(cells)), repeat=len(R)):
        rounds = [cells[c][0] for c in choice]
        lanes = [cells[c][1] for c in choice]
        if packing.grid_feasible(R, rounds, lanes, b, s, cap) and packing.grid_objective(w, rounds, lanes, b, s) == target:
            return Choice(cost, d, primitive, b, s, rounds, lanes)
    return None
