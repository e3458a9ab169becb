"""Pins for the fp64 oracle against things other than itself.

Each test names the plausible mistake it would catch.
"""
import numpy as np
import pytest
import torch

from oracle import tree_attention as ora


def _rand_tree(seed, P, R, hq, hkv, d, groups=1):
    rng = np.random.default_rng(seed)
    tb = ora.TreeBatch([P] * groups if np.isscalar(P) else P,
                       [list(R)] * groups if np.isscalar(P) else R, hq, hkv, d)
    tp, tr = int(tb.cu_p[-1]), int(tb.cu_r[-1])
    t = {
        "q_p": rng.standard_normal((tp, hq, d)), "k_p": rng.standard_normal((tp, hkv, d)),
        "v_p": rng.standard_normal((tp, hkv, d)), "do_p": rng.standard_normal((tp, hq, d)),
        "q_r": rng.standard_normal((tr, hq, d)), "k_r": rng.standard_normal((tr, hkv, d)),
        "v_r": rng.standard_normal((tr, hkv, d)), "do_r": rng.standard_normal((tr, hq, d)),
    }
    return tb, t


def _run(tb, t, **kw):
    return ora.tree_attention_fwd_bwd(tb, t["q_p"], t["k_p"], t["v_p"], t["do_p"],
                                      t["q_r"], t["k_r"], t["v_r"], t["do_r"], **kw)


# --- finite differences: wrong sign, dropped scale, missing GQA or branch sum ---
def test_gradients_match_central_differences():
    tb, t = _rand_tree(0, [5, 3], [[4, 2, 3], [1, 2]], 4, 2, 8)
    res = _run(tb, t)

    def loss(tt):
        r = _run(tb, tt, with_backward=False)
        return (r["o_p"] * t["do_p"]).sum() + (r["o_r"] * t["do_r"]).sum()

    rng = np.random.default_rng(1)
    h = 1e-6
    for name, gname in [("q_p", "dq_p"), ("k_p", "dk_p"), ("v_p", "dv_p"),
                        ("q_r", "dq_r"), ("k_r", "dk_r"), ("v_r", "dv_r")]:
        for _ in range(12):
            idx = tuple(int(rng.integers(0, s)) for s in t[name].shape)
            tp_, tm_ = dict(t), dict(t)
            tp_[name] = t[name].copy(); tp_[name][idx] += h
            tm_[name] = t[name].copy(); tm_[name][idx] -= h
            fd = (loss(tp_) - loss(tm_)) / (2 * h)
            assert abs(fd - res[gname][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, res[gname][idx])


# --- the dense tree mask over [P; R_1..R_G]: sibling leakage, wrong diagonal ---
def test_flattened_equals_dense_tree_mask():
    P, R, hq, hkv, d = 7, [5, 1, 4], 4, 2, 16
    tb, t = _rand_tree(2, [P], [R], hq, hkv, d)
    res = _run(tb, t)
    vis = ora.tree_mask(P, R)
    # mask structure: prompt column full for response rows, no sibling visibility
    assert vis[P:, :P].all() and not vis[:P, P:].any()
    assert not vis[P:P + 5, P + 5:].any() and not vis[P + 5:, P:P + 5].any()
    assert vis.sum() == ora.tri(P) + sum(r * P + ora.tri(r) for r in R)
    rep = hq // hkv
    dk = np.zeros((P + sum(R), hkv, d)); dv = np.zeros_like(dk)
    for h in range(hq):
        c = h // rep
        q = np.concatenate([t["q_p"][:, h], t["q_r"][:, h]]); k = np.concatenate([t["k_p"][:, c], t["k_r"][:, c]])
        v = np.concatenate([t["v_p"][:, c], t["v_r"][:, c]]); do = np.concatenate([t["do_p"][:, h], t["do_r"][:, h]])
        o, lse, dq, dk_h, dv_h = ora.masked_attention_fwd_bwd(q, k, v, do, vis, tb.scale)
        dk[:, c] += dk_h; dv[:, c] += dv_h
        np.testing.assert_allclose(res["o_p"][:, h], o[:P], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(res["o_r"][:, h], o[P:], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(res["lse_p"][h], lse[:P], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(res["lse_r"][h], lse[P:], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(res["dq_p"][:, h], dq[:P], rtol=1e-10, atol=1e-11)
        np.testing.assert_allclose(res["dq_r"][:, h], dq[P:], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(res["dk_p"], dk[:P], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(res["dv_p"], dv[:P], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(res["dk_r"], dk[P:], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(res["dv_r"], dv[P:], rtol=1e-10, atol=1e-11)


# --- split + merge of partial states equals the unsplit result (any split, empty parts) ---
@pytest.mark.parametrize("cuts", [[], [3], [0, 4], [2, 5, 9], [1, 2, 3, 4, 5, 6, 11]])
def test_partial_state_merge_equals_unsplit(cuts):
    P, R, d = 11, 6, 8
    tb, t = _rand_tree(3, [P], [[R]], 1, 1, d)
    res = _run(tb, t, with_backward=False)
    q = t["q_r"][:, 0]
    k = np.concatenate([t["k_p"][:, 0], t["k_r"][:, 0]]); v = np.concatenate([t["v_p"][:, 0], t["v_r"][:, 0]])
    vis = np.concatenate([np.ones((R, P), bool), np.tril(np.ones((R, R), bool))], axis=1)
    edges = [0] + cuts + [P + R]
    state = (np.full(R, -np.inf), np.zeros(R), np.zeros((R, d)))
    for a, b in zip(edges[:-1], edges[1:]):
        state = ora.merge_states(state, ora.partial_state(q, k[a:b], v[a:b], vis[:, a:b], tb.scale))
    o, lse = ora.finalize_state(state)
    np.testing.assert_allclose(o, res["o_r"][:, 0], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, res["lse_r"][0], rtol=1e-11, atol=1e-12)


def test_merge_is_associative_and_commutative():
    rng = np.random.default_rng(4)
    mk = lambda: (rng.standard_normal(5), rng.random(5) + 0.1, rng.standard_normal((5, 3)))
    a, b, c = mk(), mk(), mk()
    l = ora.finalize_state(ora.merge_states(ora.merge_states(a, b), c))
    r = ora.finalize_state(ora.merge_states(a, ora.merge_states(c, b)))
    np.testing.assert_allclose(l[0], r[0], rtol=1e-12); np.testing.assert_allclose(l[1], r[1], rtol=1e-12)


# --- G = 1 is ordinary causal attention: torch's SDPA + autograd in fp64 ---
def test_single_branch_equals_torch_sdpa():
    P, R, hq, hkv, d = 9, 6, 4, 2, 16
    tb, t = _rand_tree(5, [P], [[R]], hq, hkv, d)
    res = _run(tb, t)
    cat = lambda a, b: torch.tensor(np.concatenate([t[a], t[b]]), dtype=torch.float64)
    q = cat("q_p", "q_r").permute(1, 0, 2)[None].requires_grad_(True)
    k = cat("k_p", "k_r").permute(1, 0, 2)[None].requires_grad_(True)
    v = cat("v_p", "v_r").permute(1, 0, 2)[None].requires_grad_(True)
    do = cat("do_p", "do_r").permute(1, 0, 2)[None]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, enable_gqa=True)
    (o * do).sum().backward()
    f = lambda x: x[0].permute(1, 0, 2).detach().numpy()
    np.testing.assert_allclose(np.concatenate([res["o_p"], res["o_r"]]), f(o), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(np.concatenate([res["dq_p"], res["dq_r"]]), f(q.grad), rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(np.concatenate([res["dk_p"], res["dk_r"]]), f(k.grad), rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(np.concatenate([res["dv_p"], res["dv_r"]]), f(v.grad), rtol=1e-9, atol=1e-10)


# --- closed forms ---
def test_zero_keys_give_uniform_softmax_and_log_count():
    P, R = 6, [4, 3]
    tb, t = _rand_tree(6, [P], [R], 2, 1, 8)
    t["k_p"][:] = 0.0; t["k_r"][:] = 0.0
    res = _run(tb, t, with_backward=False)
    # inclusive diagonal: prompt row a sees a+1 keys; response row t sees P+t+1
    np.testing.assert_allclose(res["lse_p"][0], np.log(np.arange(1, P + 1)), rtol=1e-13)
    np.testing.assert_allclose(res["lse_r"][1], np.log(np.concatenate([P + 1 + np.arange(4), P + 1 + np.arange(3)])), rtol=1e-13)
    run_mean = np.cumsum(t["v_p"][:, 0], axis=0) / np.arange(1, P + 1)[:, None]
    np.testing.assert_allclose(res["o_p"][:, 0], run_mean, rtol=1e-12, atol=1e-13)
    # second branch, last row: mean of the prompt and its own 3 response values
    want = (t["v_p"][:, 0].sum(0) + t["v_r"][4:7, 0].sum(0)) / (P + 3)
    np.testing.assert_allclose(res["o_r"][6, 1], want, rtol=1e-12, atol=1e-13)


def test_first_row_and_constant_values():
    tb, t = _rand_tree(7, [5], [[3, 2]], 2, 2, 4)
    res = _run(tb, t, with_backward=False)
    np.testing.assert_allclose(res["o_p"][0], t["v_p"][0], rtol=1e-13)
    np.testing.assert_allclose(res["lse_p"][:, 0], tb.scale * (t["q_p"][0] * t["k_p"][0]).sum(-1), rtol=1e-13)
    t["v_p"][:] = 1.0; t["v_r"][:] = 1.0
    res = _run(tb, t)
    np.testing.assert_allclose(res["o_r"], 1.0, rtol=1e-13)
    np.testing.assert_allclose(res["dq_r"], 0.0, atol=1e-13)
    np.testing.assert_allclose(res["dk_p"], 0.0, atol=1e-13)


def test_identical_keys_lse():
    tb, t = _rand_tree(8, [4], [[3]], 1, 1, 8)
    t["k_p"][:] = t["k_p"][0]; t["k_r"][:] = t["k_p"][0]
    res = _run(tb, t, with_backward=False)
    s = tb.scale * (t["q_r"][:, 0] @ t["k_p"][0, 0])
    np.testing.assert_allclose(res["lse_r"][0], s + np.log(4 + 1 + np.arange(3)), rtol=1e-12)


# --- invariants of Eq. 2 and of the tree ---
def test_prompt_gradient_is_sum_over_branches_and_permutation_invariant():
    P, R, hq, hkv, d = 6, [4, 2, 5], 2, 1, 8
    tb, t = _rand_tree(9, [P], [R], hq, hkv, d)
    res = _run(tb, t)
    # per-branch trees with the prompt seed switched off, plus the prompt alone
    acc_k = np.zeros_like(res["dk_p"]); acc_v = np.zeros_like(res["dv_p"])
    off = 0
    for r in R:
        tb1 = ora.TreeBatch([P], [[r]], hq, hkv, d)
        t1 = dict(t); t1["do_p"] = np.zeros_like(t["do_p"])
        for n in ("q_r", "k_r", "v_r", "do_r"):
            t1[n] = t[n][off:off + r]
        r1 = _run(tb1, t1)
        acc_k += r1["dk_p"]; acc_v += r1["dv_p"]
        off += r
    tb0 = ora.TreeBatch([P], [[]], hq, hkv, d)
    t0 = dict(t)
    for n in ("q_r", "k_r", "v_r", "do_r"):
        t0[n] = t[n][:0]
    r0 = _run(tb0, t0)
    np.testing.assert_allclose(res["dk_p"], acc_k + r0["dk_p"], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(res["dv_p"], acc_v + r0["dv_p"], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(res["dq_p"], r0["dq_p"], rtol=1e-10, atol=1e-11)
    # permuting siblings leaves prompt gradients unchanged
    tbp = ora.TreeBatch([P], [[5, 4, 2]], hq, hkv, d)
    tp = dict(t)
    perm = np.concatenate([np.arange(6, 11), np.arange(0, 4), np.arange(4, 6)])
    for n in ("q_r", "k_r", "v_r", "do_r"):
        tp[n] = t[n][perm]
    rp = _run(tbp, tp)
    np.testing.assert_allclose(rp["dk_p"], res["dk_p"], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(rp["o_r"], res["o_r"][perm], rtol=1e-12, atol=1e-13)


def test_row_forms_match_matrix_form():
    tb, t = _rand_tree(10, [6, 4], [[3, 5], [2]], 4, 2, 8)
    res = _run(tb, t)
    for kind, tok, h in [("p", 0, 0), ("p", 7, 3), ("r", 0, 1), ("r", 7, 2), ("r", 9, 3)]:
        o, lse = ora.forward_row(tb, t["q_p"], t["k_p"], t["v_p"], t["q_r"], t["k_r"], t["v_r"], kind, tok, h)
        dq = ora.dq_row(tb, t["q_p"], t["k_p"], t["v_p"], t["do_p"], t["q_r"], t["k_r"], t["v_r"], t["do_r"], kind, tok, h)
        sfx = "_p" if kind == "p" else "_r"
        np.testing.assert_allclose(o, res["o" + sfx][tok, h], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(lse, res["lse" + sfx][h, tok], rtol=1e-12)
        np.testing.assert_allclose(dq, res["dq" + sfx][tok, h], rtol=1e-10, atol=1e-11)


def test_key_form_matches_matrix_form():
    tb, t = _rand_tree(11, [6, 4], [[3, 5], [2]], 4, 2, 8)
    res = _run(tb, t)
    for kind, tok, c in [("p", 0, 0), ("p", 5, 1), ("p", 8, 0), ("r", 0, 1), ("r", 7, 0), ("r", 9, 1)]:
        dk, dv = ora.dkv_key(tb, t["q_p"], t["k_p"], t["v_p"], t["do_p"], t["q_r"], t["k_r"], t["v_r"], t["do_r"], kind, tok, c)
        sfx = "_p" if kind == "p" else "_r"
        np.testing.assert_allclose(dk, res["dk" + sfx][tok, c], rtol=1e-10, atol=1e-11)
        np.testing.assert_allclose(dv, res["dv" + sfx][tok, c], rtol=1e-10, atol=1e-11)


def test_key_block_form_matches_key_form_and_matrix_form():
    """The row-block form (several keys, query rows a block at a time) against the per-key row form and the
    n x n matrix form, with blocks that cut through the prompt, through branches and behind the keys."""
    tb, t = _rand_tree(12, [9, 5], [[6, 1, 4], [3]], 4, 2, 8)
    res = _run(tb, t)
    a = [t[n] for n in ("q_p", "k_p", "v_p", "do_p", "q_r", "k_r", "v_r", "do_r")]
    for kind, toks, c in [("p", [0, 3, 8], 0), ("p", [9, 13], 1), ("r", [0, 5], 1), ("r", [7, 10], 0), ("r", [11, 13], 1), ("r", [6], 0)]:
        for block in (4, 256):
            dk, dv = ora.dkv_keys_block(tb, *a, kind, toks, c, block=block)
            sfx = "_p" if kind == "p" else "_r"
            for i, tok in enumerate(toks):
                k1, v1 = ora.dkv_key(tb, *a, kind, tok, c)
                np.testing.assert_allclose(dk[i], k1, rtol=1e-11, atol=1e-12)
                np.testing.assert_allclose(dv[i], v1, rtol=1e-11, atol=1e-12)
                np.testing.assert_allclose(dk[i], res["dk" + sfx][tok, c], rtol=1e-10, atol=1e-11)
                np.testing.assert_allclose(dv[i], res["dv" + sfx][tok, c], rtol=1e-10, atol=1e-11)


# --- work accounting: flattening repeats the prompt pairs G times (Sec. 1) ---
def test_redundancy_fraction():
    for G, want in [(8, 0.875), (64, 0.984375)]:
        tb = ora.TreeBatch([1000], [[10] * G], 1, 1, 8)
        pre, rep, flat = ora.valid_pairs(tb)
        assert flat - rep == G * pre
        assert abs((flat - rep - pre) / (flat - rep) - want) < 1e-12
    # reuse factors of the benchmark configurations 1-3
    for P, G, R, want in [(256, 4, 128, 1.501), (8192, 8, 2048, 2.273), (65536, 8, 1024, 6.591)]:
        pre, rep, flat = ora.valid_pairs(ora.TreeBatch([P], [[R] * G], 1, 1, 8))
        assert abs(flat / (pre + rep) - want) < 1e-3


# --------------------------------------------------------------------------- #
# Replay-grid assignment (Eq. 6): pins of the brute-force definition
def test_grid_assignment_definition_reduces_to_known_cases():
    from oracle import packing as pk
    rng = np.random.default_rng(11)
    for _ in range(12):
        U = int(rng.integers(1, 7))
        w = [int(x) for x in rng.integers(1, 40, size=U)]
        m = [1] * U
        # one lane: every round's maximum is its sum, so any assignment costs the total work
        assert pk.brute_force_grid(w, m, 2, 1, None) == sum(w)
        # no memory limit: merging rounds never lengthens the path, so several rounds buy nothing and the
        # optimum is the classical makespan on s machines (an independent exhaustive routine)
        for s in (2, 3):
            assert pk.brute_force_grid(w, m, 2, s, None) == pk.brute_force_makespan(w, s)
            assert pk.brute_force_grid(w, m, 1, s, None) == pk.brute_force_makespan(w, s)
        # at least as many cells in one round as units: the longest unit alone
        assert pk.brute_force_grid(w, m, 1, U, None) == max(w)
    # a hand-worked case with a limit of one unit per cell: 2 rounds x 2 lanes, works 5, 4, 3, 1
    # -> rounds {5,4} and {3,1} cost 5 + 3 = 8; {5,1},{4,3} costs 5 + 4 = 9; {5,3},{4,1} costs 5 + 4 = 9
    assert pk.brute_force_grid([5, 4, 3, 1], [1, 1, 1, 1], 2, 2, 1) == 8
    # five units do not fit four cells of one unit each
    assert pk.brute_force_grid([1, 1, 1, 1, 1], [1] * 5, 2, 2, 1) is None
    # a tighter limit can only lengthen the path
    w, m = [9, 7, 6, 5, 4, 2], [3, 2, 2, 1, 1, 1]
    vals = [pk.brute_force_grid(w, m, 2, 2, cap) for cap in (3, 4, 5, 10)]
    assert all(a >= b for a, b in zip(vals, vals[1:])) and vals[-1] == pk.brute_force_makespan(w, 2)


def test_grid_greedy_is_valid_and_never_beats_the_optimum():
    from oracle import packing as pk
    rng = np.random.default_rng(12)
    for _ in range(30):
        U = int(rng.integers(1, 7))
        w = [int(x) for x in rng.integers(1, 30, size=U)]
        m = [int(x) for x in rng.integers(1, 4, size=U)]
        b, s = int(rng.integers(1, 3)), int(rng.integers(1, 3))
        cap = None if rng.random() < 0.4 else int(rng.integers(3, 8))
        opt = pk.brute_force_grid(w, m, b, s, cap)
        g = pk.greedy_grid(w, m, b, s, cap)
        if g is None:
            continue  # greedy may fail to pack what an exhaustive search can
        rounds, lanes, val = g
        assert opt is not None and pk.grid_feasible(m, rounds, lanes, b, s, cap)
        assert val == pk.grid_objective(w, rounds, lanes, b, s) >= opt
