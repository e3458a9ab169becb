"""The online strategy planner (Sec. 3.4, Algorithm 1, Eq. 6-10): pins of the oracle, then the library against it.

The paper gives the form of the cost model and no constants, so the selection logic is pinned on synthetic
profiles: closed forms, the regime switch of Eq. 5, the fallback to ordinary ring CP, the memory limit that forces
rounds, and invariances.  The library is then compared with the oracle's exhaustive search on random small trees.
"""
import itertools
import time

import numpy as np
import pytest

from oracle import planner as op


def _prof(**kw):
    return op.Profile(**kw)


# ------------------------------------------------------------------------------------------ pins of the oracle
def test_closed_form_single_path():
    # P = 256, R = 128: one query tile against two prompt tiles plus its own diagonal tile = 3 tiles
    assert op.replay_tiles(256, 128) == 3 and op.replay_tiles(257, 129) == 2 * 3 + 3 and op.causal_tiles(300) == 6
    c = op.plan_tree(256, [128], 4, 4, [2], _prof(alpha_ring=1e9))
    # TreeMoveKV, one lane of both ranks: alpha_p L_P / d + alpha W / d_lane = 128 + 1.5
    assert (c.primitive, c.b, c.s, c.d) == (op.TREE_MOVE_KV, 1, 1, 2) and c.cost == 129.5
    # gamma scales the whole candidate (Eq. 7)
    c2 = op.plan_tree(256, [128], 4, 4, [2], _prof(alpha_ring=1e9, gamma_tmkv=2.0, gamma_mq=3.0))
    assert c2.cost == 259.0


def test_regime_switch_follows_the_traffic_ratio():
    """Eq. 5: with traffic as the only cost, TreeMoveKV wins while 2 (L_P + L_R) H_kv f < L_R H_q, MoveQ beyond.
    H_q = 28, H_kv = 4, d = 8 (f = 7/8): the switch is at L_P / L_R = 3."""
    comm = dict(alpha_p=0, alpha_tmkv=0, alpha_mq=0, beta_tmkv=1.0, beta_q=1.0, alpha_ring=0, lat_ring0=1e18)
    below = op.plan_tree(2900, [1000], 28, 4, [8], _prof(**comm), b_max=1)
    above = op.plan_tree(3100, [1000], 28, 4, [8], _prof(**comm), b_max=1)
    assert below.primitive == op.TREE_MOVE_KV and above.primitive == op.MOVE_Q
    assert below.cost == 2 * 3900 * 4 * 7 / 8 and above.cost == 1000 * 28
    # a reduction term moves the switch the way Eq. 5 says: T_red makes MoveQ dearer
    dearer = op.plan_tree(3100, [1000], 28, 4, [8], _prof(**comm, red1=0.2), b_max=1)
    assert dearer.primitive == op.TREE_MOVE_KV


def test_fallback_to_ring_cp_for_short_groups():
    """b = 0 is chosen when the split's fixed overheads outweigh its benefit, and not when the prompt is long."""
    prof = _prof(alpha_p=1 / 128, lat_tmkv0=50.0, lat_mq0=50.0, lat_p0=50.0)
    short = op.plan_tree(256, [128, 128], 4, 4, [1, 2], prof)
    assert short.primitive == op.RING_CP and short.b == 0
    long_ = op.plan_tree(65536, [128, 128], 4, 4, [1, 2], prof)
    assert long_.primitive != op.RING_CP          # ring CP would recompute the 64k prompt for each branch


def test_memory_limit_forces_rounds():
    """Four equal paths, one rank: a cell that holds two paths' tokens needs two rounds; without the limit one is best."""
    free = op.plan_tree(1024, [512] * 4, 4, 4, [1], _prof(alpha_ring=1e9))
    assert free.b == 1
    tight = op.plan_tree(1024, [512] * 4, 4, 4, [1], _prof(alpha_ring=1e9, mem_cap=1024 + 1024, mem_prompt=1.0, mem_resp=1.0))
    assert tight.b == 2 and sorted(np.bincount(tight.rounds).tolist()) == [2, 2]
    none = op.plan_tree(1024, [512] * 4, 4, 4, [1], _prof(alpha_ring=1e9, mem_cap=1024 + 100, mem_prompt=1.0, mem_resp=1.0,
                                                        lat_ring0=0.0))
    assert none is None or none.primitive == op.RING_CP    # not even one path fits beside the prompt


def test_candidate_set_and_invariances():
    cands = list(op.candidates(100, [10, 20, 30], [4], b_max=4))
    assert cands[0] == (4, op.RING_CP, 0, 1)
    split = [(p, b, s) for _, p, b, s in cands[1:]]
    # lanes 1 and 2 divide 4 and do not exceed G = 3 (4 lanes would leave one empty); rounds up to ceil(G / s)
    assert split == [(p, b, s) for p in (op.TREE_MOVE_KV, op.MOVE_Q) for s, bs in ((1, (1, 2, 3)), (2, (1, 2))) for b in bs]
    prof = _prof(beta_tmkv=0.01, beta_q=0.02, red0=3.0, lat_mq1=1.0, lat_tmkv1=0.5)
    a = op.plan_tree(700, [300, 150, 420], 8, 2, [2, 4], prof)
    for perm in itertools.permutations([300, 150, 420]):
        b = op.plan_tree(700, list(perm), 8, 2, [2, 4], prof)
        assert (b.cost, b.d, b.primitive, b.b, b.s) == (a.cost, a.d, a.primitive, a.b, a.s)


# ------------------------------------------------------------------------------------- the library against it
@pytest.fixture(scope="module")
def B():
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding
    return binding


def _as_dict(prof):
    return {k: getattr(prof, k) for k in prof.__dataclass_fields__}


def test_library_planner_matches_the_exhaustive_oracle(B):
    rng = np.random.default_rng(7)
    seen = set()
    for trial in range(120):
        G = int(rng.integers(0, 5))
        P = int(rng.choice([1, 100, 128, 129, 700, 4096, 20000]))
        R = [int(rng.choice([1, 64, 128, 200, 513, 3000])) for _ in range(G)]
        degrees = [int(x) for x in rng.choice([1, 2, 4, 8], size=int(rng.integers(1, 4)), replace=False)]
        u = lambda lo, hi: float(rng.uniform(lo, hi))
        prof = _prof(alpha_p=u(0, 0.1), beta_p=u(0, 0.01), lat_p0=u(0, 20), lat_p1=u(0, 2), alpha_tmkv=u(0.5, 2), beta_tmkv=u(0, 0.01),
                     lat_tmkv0=u(0, 20), lat_tmkv1=u(0, 2), alpha_mq=u(0.5, 2), beta_q=u(0, 0.005), red0=u(0, 10), red1=u(0, 0.005),
                     lat_mq0=u(0, 20), lat_mq1=u(0, 5), alpha_ring=u(0.5, 2), beta_ring=u(0, 0.01), lat_ring0=u(0, 20), lat_ring1=u(0, 2),
                     gamma_ring=u(0.8, 1.2), gamma_tmkv=u(0.8, 1.2), gamma_mq=u(0.8, 1.2))
        if trial % 3 == 0 and G:
            prof.mem_prompt, prof.mem_resp = 1.0, float(rng.choice([1.0, 2.0]))
            prof.mem_cap = float(rng.choice([P + max(R), (P + sum(R)) / 2, P / 2 + max(R), 50.0]))
        want = op.plan_tree(P, R, 8, 2, degrees, prof, b_max=3)
        if want is None:
            with pytest.raises(B.AugtreeError) as e:
                B.plan_tree(P, R, 8, 2, degrees, _as_dict(prof), b_max=3)
            assert e.value.code == -2
            continue
        got = B.plan_tree(P, R, 8, 2, degrees, _as_dict(prof), b_max=3)
        assert got["cost"] == pytest.approx(want.cost, rel=1e-12), (trial, got, want)
        assert (got["degree"], got["primitive"], got["rounds"], got["lanes"]) == (want.d, want.primitive, want.b, want.s), (trial, got, want)
        assert got["solved_exactly"]
        if want.primitive != op.RING_CP:
            # X is one of possibly several optimal placements: it must be feasible and reach the minimum of Eq. 6
            from oracle import packing
            rounds, lanes = got["X"]
            w = [op.replay_tiles(P, r) for r in R]
            cap = op.cell_token_cap(prof, want.primitive, P, want.d, want.s)
            assert packing.grid_feasible(R, rounds, lanes, want.b, want.s, cap)
            assert packing.grid_objective(w, rounds, lanes, want.b, want.s) == packing.grid_objective(w, want.rounds, want.lanes, want.b, want.s)
        seen.add(want.primitive)
    assert seen == {op.RING_CP, op.TREE_MOVE_KV, op.MOVE_Q}       # the sweep exercises all three outcomes


def test_planner_rejects_bad_arguments(B):
    with pytest.raises(B.AugtreeError) as e:
        B.plan_tree(0, [10], 4, 4, [2], {})
    assert e.value.code == -1
    with pytest.raises(B.AugtreeError) as e:
        B.plan_tree(10, [0], 4, 4, [2], {})
    assert e.value.code == -1
    with pytest.raises(B.AugtreeError) as e:
        B.plan_tree(10, [5], 4, 4, [0], {})
    assert e.value.code == -1


def test_planner_solve_time_grows_mildly(B):
    """Planner time for trees of 16 .. 8192 blocks of 512 tokens with G = 8 (the sweep of the paper's solve-time figure,
    which reports 0.018 ms to 1.70 ms on its own host): reported, and bounded loosely so that a regression to
    something super-linear shows."""
    prof = {n: 1.0 for n in ("alpha_p", "alpha_tmkv", "alpha_mq", "alpha_ring", "gamma_ring", "gamma_tmkv", "gamma_mq", "mem_resp")}
    prof.update(beta_tmkv=0.01, beta_q=0.01, red0=5.0, lat_mq1=1.0)
    times = {}
    for blocks in (16, 128, 1024, 8192):
        tokens = blocks * 512
        P, R = tokens // 2, [tokens // 16] * 8
        B.plan_tree(P, R, 28, 4, [1, 2, 4, 8], prof)
        t0 = time.perf_counter()
        for _ in range(20):
            B.plan_tree(P, R, 28, 4, [1, 2, 4, 8], prof)
        times[blocks] = (time.perf_counter() - t0) / 20 * 1e3
    print("planner ms per tree:", {k: round(v, 3) for k, v in times.items()})
    assert max(times.values()) < 50.0


def test_library_planner_above_the_exact_solver_cap(B):
    """With more units than the exact AssignGrid solver takes, the library places each candidate largest-first; the
    selection must then be Algorithm 1 over those placements: every candidate scored with Eq. 7-10 (the oracle's cost
    functions) at the greedy placement (the oracle's restatement of the rule), the cheapest kept, first on ties."""
    from oracle import packing
    rng = np.random.default_rng(23)
    for trial in range(25):
        G = int(rng.integers(9, 30))
        P = int(rng.choice([700, 4096, 20000, 65536]))
        R = [int(rng.choice([64, 200, 513, 3000, 9000])) for _ in range(G)]
        degrees = [2, 4, 8]
        u = lambda lo, hi: float(rng.uniform(lo, hi))
        prof = _prof(alpha_p=u(0, 0.1), beta_p=u(0, 0.01), lat_p0=u(0, 20), alpha_tmkv=u(0.5, 2), beta_tmkv=u(0, 0.01), lat_tmkv0=u(0, 20),
                     lat_tmkv1=u(0, 2), alpha_mq=u(0.5, 2), beta_q=u(0, 0.005), red0=u(0, 10), red1=u(0, 0.005), lat_mq0=u(0, 20),
                     lat_mq1=u(0, 5), alpha_ring=u(0.5, 2), beta_ring=u(0, 0.01), lat_ring0=u(0, 20), gamma_tmkv=u(0.8, 1.2), gamma_mq=u(0.8, 1.2))
        if trial % 2:
            prof.mem_prompt, prof.mem_resp, prof.mem_cap = 1.0, 1.0, float(P + sum(R) / 3)
        w = [op.replay_tiles(P, r) for r in R]
        best = None
        for d, primitive, b, s in op.candidates(P, R, degrees, b_max=3):
            if primitive == op.RING_CP:
                if not op.ring_feasible(prof, P, R, d):
                    continue
                cand = (op.ring_cost(prof, P, R, 8, 2, d), d, primitive, 0, 1, None)
            else:
                cap = op.cell_token_cap(prof, primitive, P, d, s)
                if cap is not None and cap < 0:
                    continue
                placed = packing.greedy_grid(w, R, b, s, cap)
                if placed is None:
                    continue
                cand = (op.split_cost(prof, primitive, P, R, 8, 2, d, b, s, placed[2]), d, primitive, b, s, placed)
            if best is None or cand[0] < best[0]:
                best = cand
        got = B.plan_tree(P, R, 8, 2, degrees, _as_dict(prof), b_max=3, exact_max_units=8)
        assert best is not None
        assert got["cost"] == pytest.approx(best[0], rel=1e-12), (trial, got, best[:5])
        assert (got["degree"], got["primitive"], got["rounds"], got["lanes"]) == best[1:5], (trial, got, best[:5])
        if best[2] != op.RING_CP:
            assert not got["solved_exactly"]
            assert (got["X"][0], got["X"][1]) == (best[5][0], best[5][1])       # the greedy rule is deterministic: same placement
