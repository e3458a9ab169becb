"""Host-side checks that need no GPU: the library loads, exports what the header
declares, validates descriptors, and its packing tables equal the independent
Python restatement bit for bit."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding as b
    return b


def test_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "augtree.h")).read()
    declared = set(re.findall(r"\b(augtree_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(binding.lib, name), name


def test_descriptor_validation(binding):
    B = binding
    with pytest.raises(B.AugtreeError) as e:
        B.Plan([16], [[4]], 3, 2, 64, device=None, n_lanes=4)
    assert e.value.code == -2                    # h_q % h_kv
    with pytest.raises(B.AugtreeError) as e:
        B.Plan([16], [[4]], 4, 2, 100, device=None, n_lanes=4)
    assert e.value.code == -2                    # head_dim not a multiple of 8
    with pytest.raises(B.AugtreeError) as e:
        B.Plan([16], [[4]], 4, 2, 136, device=None, n_lanes=4)
    assert e.value.code == -2                    # head_dim above the tile width
    assert B.Plan([16], [[4]], 4, 2, 96, device=None, n_lanes=4).head_dim == 96
    with pytest.raises(B.AugtreeError) as e:
        B.Plan([0], [[4]], 4, 2, 64, device=None, n_lanes=4)
    assert e.value.code == -1                    # empty prompt
    with pytest.raises(B.AugtreeError) as e:
        B.Plan([16], [[4, 0]], 4, 2, 64, device=None, n_lanes=4)
    assert e.value.code == -1                    # empty branch
    with pytest.raises(B.AugtreeError) as e:
        B.Plan([16], [[4]], 4, 2, 64, device=None, n_lanes=0)
    assert e.value.code == -1                    # host-only plan needs a lane count
    d = B.Desc(4, 1, 1, None, None, None, 4, 2, 64, 0.0, 0, 4, 0)   # wrong struct_size
    h = C.c_void_p()
    assert B.lib.augtree_plan_create(C.byref(d), -1, C.byref(h)) == -1
    assert B.lib.augtree_plan_create(None, -1, C.byref(h)) == -1
    assert B.lib.augtree_status_string(-5).decode().startswith("device-side wait")
    # launches on a host-only plan are refused, not crashed
    p = B.Plan([16], [[4]], 4, 2, 64, device=None, n_lanes=4)
    assert B.lib.augtree_prefill_fwd(p._h, None, None, None, None, None, None, 0, None) == -1


CASES = [
    ([256], [[128] * 4], 4, 4, 148, 1),
    ([300, 1, 129], [[5, 130, 257], [], [64]], 8, 2, 7, 1),
    ([1000, 2000], [[100, 300], [50]], 4, 1, 16, 3),
    ([8192], [[2048] * 8], 28, 4, 148, 1),
]


@pytest.mark.parametrize("pl,bl,hq,hkv,lanes,splits", CASES)
def test_tables_bit_exact(binding, pl, bl, hq, hkv, lanes, splits):
    from oracle import packing
    B = binding
    plan = B.Plan(pl, bl, hq, hkv, 128, device=None, n_lanes=lanes, kv_splits=splits)
    ref = packing.build_tables(pl, bl, hq, hkv, splits)
    assert (plan.metadata(B.TBL_CU_PROMPT) == ref["cu_p"]).all()
    assert (plan.metadata(B.TBL_CU_BRANCH) == ref["cu_b"]).all()
    assert (plan.metadata(B.TBL_CU_RESPONSE) == ref["cu_r"]).all()
    assert (plan.metadata(B.TBL_GROUP_SPLITS) == ref["group_splits"]).all()
    assert (plan.metadata(B.TBL_REPLAY_SEGMENTS).reshape(-1, 3) == ref["seg_replay"]).all()
    assert (plan.metadata(B.TBL_PREFILL_SEGMENTS).reshape(-1, 3) == ref["seg_prefill"]).all()
    for base, key, w, wf in [(B.TBL_PREFILL_FWD_ITEMS, "prefill_fwd", 12, 10), (B.TBL_REPLAY_FWD_ITEMS, "replay_fwd", 12, 10),
                             (B.TBL_REPLAY_BWD_ITEMS, "replay_bwd", 8, 7), (B.TBL_PREFILL_BWD_ITEMS, "prefill_bwd", 8, 7),
                             (B.TBL_REPLAY_DQ_ITEMS, "replay_dq", 12, 10), (B.TBL_PREFILL_DQ_ITEMS, "prefill_dq", 12, 10)]:
        items = plan.metadata(base).reshape(-1, w)
        assert items.shape == ref[key].shape and (items == ref[key]).all(), key
        ptr, order = packing.assign_lanes(ref[key][:, wf], lanes)
        assert (plan.metadata(base + 1) == ptr).all(), key
        assert (plan.metadata(base + 2) == order).all(), key
        assert sorted(order.tolist()) == list(range(len(order)))


def test_item_weights_count_visible_pairs():
    """Forward items cover every visible (query, key) pair exactly once; backward items likewise."""
    from oracle import packing, tree_attention as ora
    pl, bl, hq, hkv = [300, 129], [[5, 130, 257], [64]], 4, 2
    ref = packing.build_tables(pl, bl, hq, hkv, 2)
    tb = ora.TreeBatch(pl, bl, hq, hkv, 128)
    pre, rep, _ = ora.valid_pairs(tb)

    def fwd_pairs(items):
        tot = 0
        for it in items:
            q_pos0, rows, a_len, b_len = int(it[1]), int(it[2]), int(it[5]), int(it[7])
            tot += rows * a_len
            if b_len:
                tot += sum(q_pos0 + r + 1 for r in range(rows))
        return tot
    assert fwd_pairs(ref["prefill_fwd"]) == pre * hq
    assert fwd_pairs(ref["replay_fwd"]) == rep * hq
    assert fwd_pairs(ref["replay_dq"]) == rep * hq and fwd_pairs(ref["prefill_dq"]) == pre * hq

    def bwd_pairs(items, segs):
        tot = 0
        for it in items:
            kv_pos0, kv_rows, mode, seg0, nseg = int(it[1]), int(it[2]), int(it[4]), int(it[5]), int(it[6])
            for s in range(seg0, seg0 + nseg):
                L = int(segs[s][1])
                for k in range(kv_pos0, kv_pos0 + kv_rows):
                    tot += L if mode else max(0, L - k)
        return tot * (hq // hkv)
    assert bwd_pairs(ref["prefill_bwd"], ref["seg_prefill"]) == pre * hq
    assert bwd_pairs(ref["replay_bwd"], ref["seg_replay"]) == rep * hq


def test_greedy_assignment_within_lpt_bound():
    from oracle import packing
    rng = np.random.default_rng(0)
    for _ in range(20):
        n, m = int(rng.integers(3, 10)), int(rng.integers(2, 4))
        w = [int(x) for x in rng.integers(1, 30, n)]
        ptr, order = packing.assign_lanes(w, m)
        got = packing.makespan(w, ptr, order)
        opt = packing.brute_force_makespan(w, m)
        assert opt <= got <= opt * (4 / 3 - 1 / (3 * m)) + 1e-9


# --------------------------------------------------------------------------- #
# Replay-grid assignment (Eq. 6) against the oracle's brute-force definition
def test_assign_grid_exact_matches_brute_force(binding):
    from oracle import packing as pk
    rng = np.random.default_rng(21)
    for trial in range(60):
        U = int(rng.integers(1, 8))
        w = [int(x) for x in rng.integers(0, 50, size=U)]
        m = [int(x) for x in rng.integers(1, 5, size=U)]
        b, s = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        if (b * s) ** U > 300000:
            b = 1
        cap = None if trial % 3 == 0 else int(rng.integers(2, 9))
        want = pk.brute_force_grid(w, m, b, s, cap)
        if want is None:
            with pytest.raises(binding.AugtreeError) as e:
                binding.assign_grid(w, m, b, s, cell_cap=cap or 0)
            assert e.value.code == -2  # unsupported: no packing exists
            continue
        rounds, lanes, path, exact = binding.assign_grid(w, m, b, s, cell_cap=cap or 0)
        # the optimal value is unique; the assignment need only be valid and reach it
        assert exact and path == want
        assert all(0 <= t < b for t in rounds) and all(0 <= j < s for j in lanes)
        assert pk.grid_feasible(m, rounds, lanes, b, s, cap)
        assert pk.grid_objective(w, rounds, lanes, b, s) == want


def test_assign_grid_greedy_is_bit_exact_and_bounded(binding):
    from oracle import packing as pk
    rng = np.random.default_rng(22)
    for trial in range(40):
        U = int(rng.integers(1, 40))
        w = [int(x) for x in rng.integers(1, 1000, size=U)]
        m = [int(x) for x in rng.integers(1, 9, size=U)]
        b, s = int(rng.integers(1, 4)), int(rng.integers(1, 6))
        cap = None if trial % 2 == 0 else int(rng.integers(8, 40))
        want = pk.greedy_grid(w, m, b, s, cap)
        if U == 1:
            continue  # a single unit always takes the exact path
        if want is None:
            with pytest.raises(binding.AugtreeError):
                binding.assign_grid(w, m, b, s, cell_cap=cap or 0, exact_max_units=1)
            continue
        rounds, lanes, path, exact = binding.assign_grid(w, m, b, s, cell_cap=cap or 0, exact_max_units=1)
        assert not exact and (rounds, lanes, path) == (want[0], want[1], want[2])
        if U <= 12:  # the exact solver can only be better
            _, _, opt, ex = binding.assign_grid(w, m, b, s, cell_cap=cap or 0)
            assert ex and opt <= path
    # sixteen units, exact: the classical bound for one round, and a larger instance still answers quickly
    w = [int(x) for x in np.random.default_rng(23).integers(1, 100, size=14)]
    _, _, opt, ex = binding.assign_grid(w, None, 1, 4, exact_max_units=16)
    assert ex and max(max(w), -(-sum(w) // 4)) <= opt <= pk.makespan(w, *pk.assign_lanes(w, 4))


def test_assign_grid_rejects_bad_arguments(binding):
    with pytest.raises(binding.AugtreeError) as e:
        binding.assign_grid([1, 2], None, 0, 1)
    assert e.value.code == -1
    with pytest.raises(binding.AugtreeError) as e:
        binding.assign_grid([1, -2], None, 1, 1)
    assert e.value.code == -1
    with pytest.raises(binding.AugtreeError) as e:
        binding.assign_grid([1, 2], None, 1, 1, cell_cap=3)  # a limit needs sizes
    assert e.value.code == -1
    assert binding.assign_grid([], None, 2, 2) == ([], [], 0, True)


def test_handoff_scratch_counts_every_visible_tile_pair(binding):
    """Backward hand-off scratch = row statistics + one 32 KB dS tile per (query tile, visible KV tile, query head) of the
    larger backward call, counted here from the definition of visibility (Eq. 1)."""
    B = binding
    cdiv = lambda a, b: -(-a // b)
    for pl, bl, hq, hkv, d in [([700], [[300, 150, 420]], 8, 2, 128), ([129, 1000], [[1, 257], [640, 64, 130, 127]], 4, 4, 64),
                               ([8192], [[2048] * 8], 28, 4, 128), ([300], [[]], 4, 2, 64)]:
        plan = B.Plan(pl, bl, hq, hkv, d, device=None, n_lanes=8)
        replay = sum(cdiv(P, 128) * cdiv(r, 128) + cdiv(r, 128) * (cdiv(r, 128) + 1) // 2 for P, rs in zip(pl, bl) for r in rs)
        prefill = sum(cdiv(P, 128) * (cdiv(P, 128) + 1) // 2 for P in pl)
        extra = plan.ws_bwd_handoff_bytes - plan.ws_bwd_bytes
        assert extra == max(replay, prefill) * hq * 128 * 128 * 2, (pl, bl)
        assert plan.workspace_bytes(0) == max(plan.ws_fwd_bytes, plan.ws_bwd_bytes, 256)
        assert plan.workspace_bytes(1 << 50) >= plan.ws_bwd_handoff_bytes


def test_handoff_is_switched_off_when_a_slot_index_would_overflow(binding):
    """Slot indices are 32-bit tensor-map coordinates: a plan with more than 2^31 (tile pair, head) slots reports
    SIZE_MAX, so that no scratch size can select the hand-off path."""
    B = binding
    plan = B.Plan([1_200_000], [[]], 64, 8, 128, device=None, n_lanes=148)
    tiles = -(-1_200_000 // 128)
    assert tiles * (tiles + 1) // 2 * 64 > 2 ** 31
    assert plan.ws_bwd_handoff_bytes == 2 ** 64 - 1
    assert plan.workspace_bytes(2 ** 62) == max(plan.ws_fwd_bytes, plan.ws_bwd_bytes, 256)
