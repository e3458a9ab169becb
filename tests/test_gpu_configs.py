"""GPU parity on the shapes of the five benchmark configurations.

Scaled-down versions (lengths and head counts reduced so that the fp64 oracle finishes in seconds, same
structure: GQA ratio, group and branch counts, length distributions) are compared element by element.
Configuration 2 is also run at its full size, in the launch configuration the benchmark times, and checked
on sampled query rows and keys that the oracle can compute one by one, plus properties that hold at any size.
"""
import numpy as np
import pytest
import torch

from oracle import tree_attention as ora
from paper_2609_33133_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding
    return binding


def _scaled(index, scale, h_q, h_kv):
    w = wl.config(index, scale_down=scale)
    return wl.Workload(w.name + f"/{scale}", w.prompt_len, w.branch_len, h_q, h_kv, w.head_dim, w.seed, extra=w.extra)


SCALED = [
    (_scaled(2, 8, 14, 2), 0),      # P=1024, 8 x 256, GQA 7:1
    (_scaled(3, 32, 8, 2), 4),      # 2 groups, P=2048, 8 x 32: prompt-dominated, 4 prompt-KV shards + merge
    (_scaled(4, 16, 8, 2), 0),      # 4 groups, P=64, 16 log-normal branches each: response-dominated
    (_scaled(5, 16, 8, 2), 0),      # 32 ragged groups
]


@pytest.mark.parametrize("w,splits", SCALED, ids=[w.name for w, _ in SCALED])
def test_scaled_configs_match_oracle(B, w, splits):
    t = wl.make_tensors(w)
    got, plan = pu.run_gpu(B, w, t, kv_splits=splits)
    if splits:
        assert plan.metadata(B.TBL_GROUP_SPLITS).max() == splits
    pu.assert_parity(got, pu.run_oracle(w, t))


def test_config2_full_size_sampled(B):
    """Full-size 7B-shaped layer, default plan (the one bench.py times): sampled rows and keys against the oracle."""
    w = wl.config(2)
    t = wl.make_tensors(w)
    got, _ = pu.run_gpu(B, w, t, flags=B.FLAG_ZERO_PROMPT_GRAD)
    assert all(np.isfinite(v).all() for v in got.values())
    tb = ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim)
    f = {k: v.float().numpy() for k, v in t.items()}
    rng = np.random.default_rng(5)
    # query rows: first / last rows of tiles, ragged positions, all head groups
    rows = [("p", 0, 0), ("p", 127, 27), ("p", 128, 5), ("p", 8191, 13), ("r", 0, 1), ("r", 2047, 26), ("r", 2048, 7), ("r", 16383, 20)]
    rows += [("p", int(rng.integers(0, 8192)), int(rng.integers(0, 28))) for _ in range(8)]
    rows += [("r", int(rng.integers(0, 16384)), int(rng.integers(0, 28))) for _ in range(12)]
    for kind, tok, h in rows:
        o, lse = ora.forward_row(tb, f["q_p"], f["k_p"], f["v_p"], f["q_r"], f["k_r"], f["v_r"], kind, tok, h)
        dq = ora.dq_row(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], kind, tok, h)
        sfx = "_p" if kind == "p" else "_r"
        assert abs(got["lse" + sfx][h, tok] - lse) <= pu.LSE_ABS, (kind, tok, h)
        assert np.abs(got["o" + sfx][tok, h] - o).max() <= pu.MAX_ABS, (kind, tok, h)
        assert np.linalg.norm(got["o" + sfx][tok, h] - o) <= 2 * pu.REL_L2 * np.linalg.norm(o) + 1e-3, (kind, tok, h)
        assert np.abs(got["dq" + sfx][tok, h] - dq).max() <= pu.MAX_ABS, (kind, tok, h)
        assert np.linalg.norm(got["dq" + sfx][tok, h] - dq) <= 2 * pu.REL_L2 * np.linalg.norm(dq) + 1e-3, (kind, tok, h)
    # keys that few rows see (ends of branches): dK, dV against the per-key oracle form
    for tok, c in [(2047, 0), (2040, 3), (16383, 1), (16370, 2), (4090, 1)]:
        dk, dv = ora.dkv_key(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], "r", tok, c)
        assert np.abs(got["dk_r"][tok, c] - dk).max() <= pu.MAX_ABS and np.abs(got["dv_r"][tok, c] - dv).max() <= pu.MAX_ABS
        assert np.linalg.norm(got["dv_r"][tok, c] - dv) <= 2 * pu.REL_L2 * np.linalg.norm(dv) + 2e-3
    # properties that hold at any size: every row's softmax sums to one, so V = 1 gives O = 1 and zero dQ/dK
    t1 = dict(t)
    t1["v_p"] = torch.ones_like(t["v_p"]); t1["v_r"] = torch.ones_like(t["v_r"])
    got1, _ = pu.run_gpu(B, w, t1, flags=B.FLAG_ZERO_PROMPT_GRAD)
    assert np.abs(got1["o_r"] - 1).max() <= 2 ** -7 and np.abs(got1["o_p"] - 1).max() <= 2 ** -7
    # dS = P * (dP - delta) vanishes up to the bf16 rounding of O inside delta
    assert np.abs(got1["dq_r"]).max() <= 0.05 and np.abs(got1["dk_p"]).max() <= 0.5
    # LSE does not depend on V
    assert np.array_equal(got1["lse_r"], got["lse_r"]) and np.array_equal(got1["lse_p"], got["lse_p"])


class _DeviceRows:
    """Indexable view of a device tensor that hands the oracle's row forms fp32 host copies of just the
    slices they ask for (the full-size tensors of configurations 3-5 are too large to widen on the host)."""

    def __init__(self, t):
        self.t = t

    def __getitem__(self, idx):
        return self.t[idx].float().cpu().numpy()


@pytest.mark.parametrize("index", [3, 4, 5])
def test_large_configs_full_size_sampled(B, index):
    """Configurations 3-5 at full size (0.15 M, 0.65 M and 0.94 M tokens; the query tensors of 4 and 5 have more
    than 2^31 elements), in the plan bench.py times: sampled query rows and keys against the oracle's row forms,
    among them the first and last tokens, tokens either side of element offset 2^31, and ends of branches."""
    w = wl.config(index)
    splits = 4 if w.extra.get("force_split") else 0
    t = wl.make_tensors(w, device="cuda")
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0, flags=B.FLAG_ZERO_PROMPT_GRAD, kv_splits=splits)
    out = B.alloc_outputs(plan)
    B.run_forward_backward(plan, t, out)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    tb = ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim)
    f = {k: _DeviceRows(v) for k, v in t.items()}
    host = lambda x: x.float().cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(40 + index)
    tp, tr = w.total_prompt, w.total_response
    edge = 2 ** 31 // (w.h_q * w.head_dim)  # first token whose element offset in a query-sized tensor passes 2^31
    rows = [("p", 0, 0), ("p", tp - 1, w.h_q - 1), ("r", 0, 1), ("r", tr - 1, w.h_q - 1)]
    rows += [("r", tok, int(rng.integers(0, w.h_q))) for tok in (edge - 1, edge, edge + 1, 2 * edge) if tok < tr]
    rows += [("p", int(rng.integers(0, tp)), int(rng.integers(0, w.h_q))) for _ in range(4)]
    rows += [("r", int(rng.integers(0, tr)), int(rng.integers(0, w.h_q))) for _ in range(8)]
    for kind, tok, h in rows:
        o, lse = ora.forward_row(tb, f["q_p"], f["k_p"], f["v_p"], f["q_r"], f["k_r"], f["v_r"], kind, tok, h)
        dq = ora.dq_row(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], kind, tok, h)
        sfx = "_p" if kind == "p" else "_r"
        g_lse, g_o, g_dq = float(out["lse" + sfx][h, tok]), host(out["o" + sfx][tok, h]), host(out["dq" + sfx][tok, h])
        assert abs(g_lse - lse) <= pu.LSE_ABS, (kind, tok, h)
        assert np.abs(g_o - o).max() <= pu.MAX_ABS, (kind, tok, h)
        assert np.linalg.norm(g_o - o) <= 2 * pu.REL_L2 * np.linalg.norm(o) + 1e-3, (kind, tok, h)
        assert np.abs(g_dq - dq).max() <= pu.MAX_ABS, (kind, tok, h)
        assert np.linalg.norm(g_dq - dq) <= 2 * pu.REL_L2 * np.linalg.norm(dq) + 1e-3, (kind, tok, h)
    # response keys near the end of a branch (few rows see them): the last branch, one in the middle, the first
    cu_r = tb.cu_r
    for b in (len(cu_r) - 2, (len(cu_r) - 1) // 2, 0):
        for back in (1, 9):
            tok = int(cu_r[b + 1]) - back
            if tok < int(cu_r[b]):
                continue
            c = int(rng.integers(0, w.h_kv))
            dk, dv = ora.dkv_key(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], "r", tok, c)
            g_dk, g_dv = host(out["dk_r"][tok, c]), host(out["dv_r"][tok, c])
            assert np.abs(g_dk - dk).max() <= pu.MAX_ABS and np.abs(g_dv - dv).max() <= pu.MAX_ABS, (b, tok, c)
            assert np.linalg.norm(g_dv - dv) <= 2 * pu.REL_L2 * np.linalg.norm(dv) + 2e-3, (b, tok, c)
    # a prompt key (Eq. 2: summed over every branch and query head of its group): the last prompt token of the
    # group whose branches are shortest, so that the per-key oracle form stays affordable
    cost = [sum(bl) * (p + max(bl)) for p, bl in zip(w.prompt_len, w.branch_len)]
    g = int(np.argmin(cost))
    if cost[g] * (w.h_q // w.h_kv) * w.head_dim <= 4e10:
        tok = int(tb.cu_p[g + 1]) - 1
        dk, dv = ora.dkv_key(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], "p", tok, 0)
        g_dk, g_dv = host(out["dk_p"][tok, 0]), host(out["dv_p"][tok, 0])
        bound = max(pu.MAX_ABS, pu.BF16_UNIT_ROUNDOFF * max(np.abs(dk).max(), np.abs(dv).max()))
        assert np.abs(g_dk - dk).max() <= bound and np.abs(g_dv - dv).max() <= bound, (g, tok)
        assert np.linalg.norm(g_dv - dv) <= 2 * pu.REL_L2 * np.linalg.norm(dv) + 2e-3, (g, tok)
    # every output finite (checked on the device)
    for k, v in out.items():
        if k != "ws":
            assert bool(torch.isfinite(v).all()), k
