"""Seeded workload generator: determinism, ranges and the token totals of the five configurations."""
import numpy as np

from paper_2609_33133_b200 import workloads as wl
from oracle import tree_attention as ora


def test_golden_redundancy_matches_pair_count():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "prompt_redundancy.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        G, pct = line.split()
        G, pct = int(G), float(pct)
        pre, rep, flat = ora.valid_pairs(ora.TreeBatch([4096], [[1] * G], 1, 1, 8))
        redundant = (flat - rep - pre) / (flat - rep)
        assert abs(100 * redundant - pct) < 0.05


def test_fixed_configs():
    w = wl.config(2)
    assert (w.total_prompt, w.total_response, w.h_q, w.h_kv, w.head_dim) == (8192, 16384, 28, 4, 128)
    w = wl.config(3)
    assert w.n_groups == 2 and w.total_prompt == 131072 and w.total_response == 16384


def test_lognormal_configs_are_deterministic_and_clipped():
    a, b = wl.config(4), wl.config(4)
    assert a.branch_len == b.branch_len and len(a.branch_len) == 4 and all(len(x) == 16 for x in a.branch_len)
    assert all(512 <= r <= 32768 for x in a.branch_len for r in x)
    med = np.median([r for x in a.branch_len for r in x])
    assert 5000 < med < 13000
    c = wl.config(5)
    assert c.n_groups == 32 and all(256 <= p <= 32768 for p in c.prompt_len)
    assert all(64 <= r <= 16384 for x in c.branch_len for r in x)
    tot = c.total_prompt + c.total_response
    assert 500_000 < tot < 1_300_000          # the distributions give ~0.8-0.9 M tokens, not 256 K
    pre = wl.config5_prefix_256k()
    assert pre.total_prompt + pre.total_response >= 262144
    assert pre.n_groups < 32


def test_counter_normal_moments():
    rng = wl.CounterNormal(123)
    z = np.array([rng.normal() for _ in range(20000)])
    assert abs(z.mean()) < 0.03 and abs(z.std() - 1) < 0.03


def test_tensors_seeded_and_flattening_is_data_movement():
    w = wl.config(1, scale_down=8)
    t1, t2 = wl.make_tensors(w), wl.make_tensors(w)
    assert all((t1[n] == t2[n]).all() for n in wl.TENSOR_NAMES)
    f = wl.flatten_tensors(w, t1)
    fw = w.flattened()
    assert f["q_p"].shape[0] == sum(fw.prompt_len) == 4 * (32 + 16)
    assert (f["k_p"][:32] == t1["k_p"]).all() and (f["k_p"][48:80] == t1["k_p"]).all()
    assert (f["do_p"][:32].float() * 4 == t1["do_p"].float()).all()
