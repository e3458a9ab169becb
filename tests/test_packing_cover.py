"""Pins of the pack-and-schedule tables by the mathematics, with no knowledge of how they were produced.

Every work item is expanded, from its documented fields alone, into the explicit (query token, key token,
query head) triples it makes a kernel visit.  For each of the six schedules the multiset of triples must equal
the tree mask of Eq. 1 (shared prompt column + block-diagonal causal branches) exactly once per pair; an
item's weight must be the number of 128 x 128 tiles it visits, which is its count of tiles holding at least
one visible pair (plus, for a forward unit of two query tiles, the one diagonal tile its first query tile sees
nothing of); each prompt-KV tile must have a single owner in the replay backward (the fixed-order sum of Eq. 2);
and a query-side item must point at the row-statistics tile that holds its rows.  The same checks run on the
oracle's restatement (oracle/packing.py) and on the library's own tables, so neither is pinned by the other.
"""
import numpy as np
import pytest

from oracle import packing
from oracle import tree_attention as ora

T = 128

CASES = [
    # prompt_len, branch_len, h_q, h_kv, kv_splits
    ([300, 1, 129], [[5, 130, 257], [], [64]], 4, 2, 1),      # ragged, a group with no branch, GQA 2:1
    ([1000, 200], [[100, 300], [50]], 4, 1, 3),               # prompt-KV shards, GQA 4:1
    ([260], [[257, 256, 1]], 2, 2, 2),                        # lengths either side of the tile edges, shards
    ([400, 131], [[], []], 2, 1, 1),                          # the flattened baseline's shape: prompts only
]


def _expected(pl, bl, hq):
    """Visibility over [all prompt tokens; all response tokens] x the same, from the tree mask of each group."""
    tb = ora.TreeBatch(pl, bl, hq, 1, 128)
    tp, tr = int(tb.cu_p[-1]), int(tb.cu_r[-1])
    vis = np.zeros((tp + tr, tp + tr), dtype=np.int64)
    for g, P in enumerate(pl):
        p0 = int(tb.cu_p[g])
        m = ora.tree_mask(P, bl[g])
        idx = list(range(p0, p0 + P))
        for i in range(len(bl[g])):
            b = int(tb.cu_b[g]) + i
            idx += list(range(tp + int(tb.cu_r[b]), tp + int(tb.cu_r[b + 1])))
        idx = np.asarray(idx)
        vis[np.ix_(idx, idx)] = m
    return vis, tp, tr


def _tile_count(block):
    """Number of 128 x 128 tiles of a visibility block (rows from a tile-aligned query start, columns from a
    tile-aligned key start) that hold at least one visible pair."""
    n = 0
    for i in range(0, block.shape[0], T):
        for j in range(0, block.shape[1], T):
            n += bool(block[i:i + T, j:j + T].any())
    return n


def _expand_forward(items, q_is_prompt, tp, tr, hq, rep, seg, sharded_ok):
    """Coverage counts [hq, tokens, tokens] of forward-type items (forward units and query-side backward units)."""
    cov = np.zeros((hq, tp + tr, tp + tr), dtype=np.int64)
    q_base = 0 if q_is_prompt else tp
    for it in items:
        q_tok0, q_pos0, q_rows, head, a_tok0, a_len, b_tok0, b_len, f8, n_splits, weight, kvh = [int(x) for x in it]
        assert kvh == head // rep                                   # GQA mapping
        assert 1 <= q_rows and q_pos0 % T == 0
        if not sharded_ok:
            assert n_splits == 1
        rows = q_base + q_tok0 + np.arange(q_rows)
        block = np.zeros((q_rows, 0), dtype=bool)
        if a_len:                                                   # unmasked range: keys of the prompt tensor
            cov[head][np.ix_(rows, a_tok0 + np.arange(a_len))] += 1
            block = np.ones((q_rows, -(-a_len // T) * T), dtype=bool)
            block[:, a_len:] = False
        if b_len:                                                   # causal range: keys of the queries' own tensor
            pos = q_pos0 + np.arange(q_rows)
            assert b_len == pos[-1] + 1                             # clipped to what the last row sees
            see = np.arange(b_len)[None, :] <= pos[:, None]
            r, c = np.nonzero(see)
            np.add.at(cov[head], (rows[r], q_base + b_tok0 + c), 1)
            pad = np.zeros((q_rows, -(-b_len // T) * T), dtype=bool)
            pad[:, :b_len] = see
            block = np.concatenate([block, pad], axis=1)
        visited = (block.shape[1] // T) * -(-q_rows // T)
        valid = _tile_count(block)
        assert weight == visited, (it, visited)
        if q_rows <= T:
            assert valid == visited                                 # one query tile: weight = valid tile count
        else:
            assert valid <= visited <= valid + 1                    # two tiles: the first sees nothing of the last key tile
        if seg is not None:                                         # query-side unit: field 8 = its row-statistics tile
            s = [x for x in seg if x[0] <= q_tok0 < x[0] + x[1]]
            assert len(s) == 1 and (q_tok0 - s[0][0]) % T == 0
            assert f8 == s[0][2] + (q_tok0 - s[0][0]) // T
            assert q_rows == min(T, s[0][0] + s[0][1] - q_tok0)
    return cov


def _expand_backward(items, seg, keys_are_prompt_in_mode0, tp, tr, hq, rep):
    cov = np.zeros((hq, tp + tr, tp + tr), dtype=np.int64)
    owners = {}
    for n, it in enumerate(items):
        kv_tok0, kv_pos0, kv_rows, kvh, mode, seg0, nseg, weight = [int(x) for x in it]
        assert 1 <= kv_rows <= T and kv_pos0 % T == 0
        key_base = 0 if (mode == 1 or keys_are_prompt_in_mode0) else tp
        q_base = 0 if keys_are_prompt_in_mode0 else tp            # prefill call: queries are prompt tokens
        keys = key_base + kv_tok0 + np.arange(kv_rows)
        visits = 0
        for s in range(seg0, seg0 + nseg):
            s_tok0, s_len, _ = [int(x) for x in seg[s]]
            a = np.arange(s_len)
            see = np.ones((s_len, kv_rows), dtype=bool) if mode else (a[:, None] >= kv_pos0 + np.arange(kv_rows)[None, :])
            r, c = np.nonzero(see)
            for h in range(kvh * rep, (kvh + 1) * rep):
                np.add.at(cov[h], (q_base + s_tok0 + r, keys[c]), 1)
            visits += sum(bool(see[i:i + T].any()) for i in range(0, s_len, T)) * rep
        assert weight == visits, (it, visits)                       # weight = valid (query tile, head) visits
        if mode == 1:
            assert (kv_tok0, kvh) not in owners                     # one owner per prompt-KV tile and KV head (Eq. 2)
            owners[(kv_tok0, kvh)] = n
    return cov, owners


def _check_tables(tab, pl, bl, hq, hkv):
    rep = hq // hkv
    vis, tp, tr = _expected(pl, bl, hq)
    want_prefill = np.zeros_like(vis); want_prefill[:tp, :tp] = vis[:tp, :tp]
    want_replay = np.zeros_like(vis); want_replay[tp:, :] = vis[tp:, :]
    seg_r, seg_p = tab["seg_replay"].reshape(-1, 3).tolist(), tab["seg_prefill"].reshape(-1, 3).tolist()
    for name, cov in [
        ("prefill_fwd", _expand_forward(tab["prefill_fwd"], True, tp, tr, hq, rep, None, False)),
        ("prefill_dq", _expand_forward(tab["prefill_dq"], True, tp, tr, hq, rep, seg_p, False)),
        ("prefill_bwd", _expand_backward(tab["prefill_bwd"], seg_p, True, tp, tr, hq, rep)[0]),
    ]:
        for h in range(hq):
            assert np.array_equal(cov[h], want_prefill), (name, h)
    rb_cov, owners = _expand_backward(tab["replay_bwd"], seg_r, False, tp, tr, hq, rep)
    for name, cov in [
        ("replay_fwd", _expand_forward(tab["replay_fwd"], False, tp, tr, hq, rep, None, True)),
        ("replay_dq", _expand_forward(tab["replay_dq"], False, tp, tr, hq, rep, seg_r, False)),
        ("replay_bwd", rb_cov),
    ]:
        for h in range(hq):
            assert np.array_equal(cov[h], want_replay), (name, h)
    # every prompt-KV tile of a group that has branches is owned, once per KV head
    n_owned = sum(-(-P // T) for P, b in zip(pl, bl) if b) * hkv
    assert len(owners) == n_owned
    # segments: tiles numbered consecutively, segment by segment
    for seg, lens in ((seg_r, [r for b in bl for r in b]), (seg_p, pl)):
        tile = tok = 0
        assert len(seg) == len(lens)
        for (s_tok0, s_len, s_tile0), L in zip(seg, lens):
            assert (s_tok0, s_len, s_tile0) == (tok, L, tile)
            tok += L; tile += -(-L // T)


@pytest.mark.parametrize("pl,bl,hq,hkv,splits", CASES)
def test_oracle_tables_cover_the_tree_mask_exactly_once(pl, bl, hq, hkv, splits):
    _check_tables(packing.build_tables(pl, bl, hq, hkv, splits), pl, bl, hq, hkv)


@pytest.mark.parametrize("pl,bl,hq,hkv,splits", CASES)
def test_library_tables_cover_the_tree_mask_exactly_once(pl, bl, hq, hkv, splits):
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding as B
    plan = B.Plan(pl, bl, hq, hkv, 128, device=None, n_lanes=5, kv_splits=splits)
    tab = {"seg_replay": plan.metadata(B.TBL_REPLAY_SEGMENTS), "seg_prefill": plan.metadata(B.TBL_PREFILL_SEGMENTS)}
    for key, base, width in [("prefill_fwd", B.TBL_PREFILL_FWD_ITEMS, 12), ("replay_fwd", B.TBL_REPLAY_FWD_ITEMS, 12),
                             ("replay_bwd", B.TBL_REPLAY_BWD_ITEMS, 8), ("prefill_bwd", B.TBL_PREFILL_BWD_ITEMS, 8),
                             ("replay_dq", B.TBL_REPLAY_DQ_ITEMS, 12), ("prefill_dq", B.TBL_PREFILL_DQ_ITEMS, 12)]:
        items = plan.metadata(base).reshape(-1, width)
        order = plan.metadata(base + 2)
        ptr = plan.metadata(base + 1)
        # the lanes partition the items: what the kernels run is exactly the item list
        assert sorted(order.tolist()) == list(range(len(items))) and ptr[0] == 0 and ptr[-1] == len(items)
        assert (np.diff(ptr) >= 0).all()
        tab[key] = items
    _check_tables(tab, pl, bl, hq, hkv)


def test_sharded_forward_items_partition_the_prompt_range():
    """With prompt-KV shards, the shards of one (query unit, head) split the prompt keys into disjoint runs of
    whole tiles and exactly one of them carries the causal range (so the merged state sees every key once)."""
    tab = packing.build_tables([1000], [[300]], 2, 1, 3)
    by_unit = {}
    for it in tab["replay_fwd"]:
        by_unit.setdefault((int(it[0]), int(it[3])), []).append([int(x) for x in it])
    for unit, its in by_unit.items():
        assert [x[8] for x in its] == list(range(its[0][9]))
        assert sum(1 for x in its if x[7] > 0) == 1
        edges = sorted((x[4], x[4] + x[5]) for x in its)
        assert edges[0][0] == 0 and edges[-1][1] == 1000
        assert all(a[1] == b[0] and a[1] % T == 0 for a, b in zip(edges, edges[1:]))
