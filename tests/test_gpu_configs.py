"""GPU parity on the shapes of the five benchmark configurations.

Scaled-down versions (lengths and head counts reduced so that the fp64 oracle finishes in seconds, same
structure: GQA ratio, group and branch counts, length distributions) are compared element by element.
At full size, in the launch configuration bench.py times:
  * configuration 2: one whole KV-head group (its 7 query heads, all 24 576 rows) element by element,
    including the full prompt-KV gradient of that head (the many-to-one sum of Eq. 2), plus sampled rows of
    the other heads and properties that hold at any size;
  * configurations 3-5: sampled query rows, response keys at the ends of branches, and prompt keys (tile-edge,
    middle and last keys of one group and KV head: Eq. 2 over every branch and query head of the group)
    against the oracle's row and row-block forms.
Sampled checks assert the stated bounds: every sampled element within 2e-2 (LSE 1e-3) and the relative L2
error over the sample within 5e-3.
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
    exceptions = None
    if w.name.startswith("cfg5"):
        # The scaled-down mixed batch has a 17-token prompt under 1100 response rows x 4 query heads.  Its
        # prompt-KV gradient (Eq. 2) is a sum of ~4400 products per element whose operands P and dS are bf16:
        # the absolute error grows like sqrt(rows) x term size whatever the (cancelling) result.  Measured:
        # one element of 1.4 M at 2.03e-2 (|ref| up to 9.9, rel-L2 1.8e-3).  Bound for this case only: one bf16
        # unit roundoff (2^-8) of the tensor's largest magnitude.
        ref = pu.run_oracle(w, t)
        exceptions = {k: {"max_abs": max(pu.MAX_ABS, 2.0 ** -8 * float(np.abs(ref[k]).max()))} for k in ("dk_p", "dv_p")}
        pu.assert_parity(got, ref, exceptions=exceptions)
        return
    pu.assert_parity(got, pu.run_oracle(w, t))


def _sample_rows(tb, f, got, rows, get=lambda x: x):
    """Sampled query rows (kind, token, head): O, LSE and dQ against the oracle's row forms."""
    acc = {k: pu.SampledError(k) for k in ("o_p", "o_r", "dq_p", "dq_r")}
    for kind, tok, h in rows:
        o, lse = ora.forward_row(tb, f["q_p"], f["k_p"], f["v_p"], f["q_r"], f["k_r"], f["v_r"], kind, tok, h)
        dq = ora.dq_row(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], kind, tok, h)
        sfx = "_p" if kind == "p" else "_r"
        assert abs(float(got["lse" + sfx][h, tok]) - lse) <= pu.LSE_ABS, (kind, tok, h)
        acc["o" + sfx].add(get(got["o" + sfx][tok, h]), o, (kind, tok, h))
        acc["dq" + sfx].add(get(got["dq" + sfx][tok, h]), dq, (kind, tok, h))
    return {k: a.check() for k, a in acc.items() if a.n}


def test_config2_full_size_one_kv_head_group(B):
    """Full-size 7B-shaped layer, default plan (the one bench.py times).  KV head 2 with its seven query heads
    is compared with the oracle element by element over all 24 576 rows: O, LSE, dQ, dK_R, dV_R and the whole
    prompt-KV gradient dK_P, dV_P of that head, i.e. the sum over 8 branches x 7 heads x 16 query tiles plus
    the prefill's own part (Eq. 2).  The other heads are sampled."""
    w = wl.config(2)
    t = wl.make_tensors(w)
    got, _ = pu.run_gpu(B, w, t, flags=B.FLAG_ZERO_PROMPT_GRAD)
    assert all(np.isfinite(v).all() for v in got.values())
    c, rep = 2, w.h_q // w.h_kv
    hs = slice(c * rep, (c + 1) * rep)
    sub = wl.Workload("cfg2-kv-head-2", w.prompt_len, w.branch_len, rep, 1, w.head_dim, w.seed)
    t_sub = {k: (v[:, hs] if v.shape[1] == w.h_q else v[:, c:c + 1]).contiguous() for k, v in t.items()}
    ref = pu.run_oracle(sub, t_sub)
    got_sub = {}
    for k, v in got.items():
        if k.startswith("lse"):
            got_sub[k] = v[hs]
        else:
            got_sub[k] = v[:, hs] if v.shape[1] == w.h_q else v[:, c:c + 1]
    rows = pu.assert_parity(got_sub, ref)
    print("cfg2 KV head 2, (rel-L2, max-abs) per tensor:", {k: (round(r[0], 5), round(r[1], 5)) for k, r in rows.items()})
    # sampled rows of the other heads: first / last rows of tiles, ragged positions
    tb = ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim)
    f = {k: v.float().numpy() for k, v in t.items()}
    rng = np.random.default_rng(5)
    samples = [("p", 0, 0), ("p", 127, 27), ("p", 128, 5), ("p", 8191, 13), ("r", 0, 1), ("r", 2047, 26), ("r", 2048, 7), ("r", 16383, 20)]
    samples += [("p", int(rng.integers(0, 8192)), int(rng.integers(0, 28))) for _ in range(6)]
    samples += [("r", int(rng.integers(0, 16384)), int(rng.integers(0, 28))) for _ in range(10)]
    _sample_rows(tb, f, got, samples)
    # keys of other KV heads: ends of branches (few rows see them) and prompt keys (every row sees them)
    for kind, toks, cc in [("r", [2040, 2047], 0), ("r", [16370, 16383], 1), ("r", [4090], 3), ("p", [0, 127, 128, 8191], 0)]:
        dk, dv = ora.dkv_keys_block(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], kind, toks, cc)
        sfx = "_p" if kind == "p" else "_r"
        a_k, a_v = pu.SampledError("dk" + sfx), pu.SampledError("dv" + sfx)
        for i, tok in enumerate(toks):
            a_k.add(got["dk" + sfx][tok, cc], dk[i], (kind, tok, cc))
            a_v.add(got["dv" + sfx][tok, cc], dv[i], (kind, tok, cc))
        a_k.check(); a_v.check()


def test_config2_full_size_handoff_against_recompute(B):
    """Full-size 7B-shaped layer on the dS hand-off path (8.5 GB of scratch, 318 k stored tiles, slot arithmetic at
    scale) against the recomputing path that the test above holds to the oracle: the key-side results bit for bit, dQ
    (from the stored dS tiles instead of the query-side kernel's own recomputation) to one bf16 step."""
    w = wl.config(2)
    t = wl.make_tensors(w)
    re_, _ = pu.run_gpu(B, w, t, flags=B.FLAG_ZERO_PROMPT_GRAD, handoff_limit=0)
    ho_, plan = pu.run_gpu(B, w, t, flags=B.FLAG_ZERO_PROMPT_GRAD, handoff_limit=1 << 40)
    assert plan.ws_bwd_handoff_bytes > 8e9
    for k in ("o_p", "lse_p", "o_r", "lse_r", "dk_r", "dv_r", "dk_p", "dv_p"):
        assert np.array_equal(re_[k], ho_[k]), k
    for k in ("dq_p", "dq_r"):
        diff = np.abs(re_[k] - ho_[k])
        # the recomputing kernel rounds its own dS (its exponentials fall on the polynomial / special-function paths
        # in a different pattern), so a few per cent of the dS values differ by a bf16 step between the paths; the dQ
        # sums then land one bf16 step apart on a minority of the elements (measured: 10-12 %, relative L2 7e-4 to 1e-3)
        assert diff.max() <= 2.0 ** -7 * max(1.0, np.abs(re_[k]).max()), (k, diff.max())
        rel = np.linalg.norm(diff.ravel()) / np.linalg.norm(re_[k].ravel())
        print(k, "differing elements", float((diff > 0).mean()), "relative L2 of the difference", float(rel))
        assert (diff > 0).mean() < 0.25 and rel <= 2e-3, (k, (diff > 0).mean(), rel)
    for kind in range(6):
        done, want = plan.items_completed(kind)
        assert done == want


def test_config2_full_size_properties(B):
    """Properties that hold at any size, on the full-size 7B-shaped layer."""
    w = wl.config(2)
    t = wl.make_tensors(w)
    got, _ = pu.run_gpu(B, w, t, flags=B.FLAG_ZERO_PROMPT_GRAD)
    # every row's softmax sums to one, so V = 1 gives O = 1, and dS = P (dP - delta) vanishes up to the bf16
    # rounding of O inside delta: dQ = dK = 0
    t1 = dict(t)
    t1["v_p"] = torch.ones_like(t["v_p"]); t1["v_r"] = torch.ones_like(t["v_r"])
    got1, _ = pu.run_gpu(B, w, t1, flags=B.FLAG_ZERO_PROMPT_GRAD)
    assert np.abs(got1["o_r"] - 1).max() <= 2 ** -7 and np.abs(got1["o_p"] - 1).max() <= 2 ** -7
    assert np.abs(got1["dq_r"]).max() <= 0.05 and np.abs(got1["dq_p"]).max() <= 0.05
    # LSE does not depend on V
    assert np.array_equal(got1["lse_r"], got["lse_r"]) and np.array_equal(got1["lse_p"], got["lse_p"])
    # every gradient is linear in dO: doubling dO doubles it bit for bit (a power of two commutes with every
    # rounding on the path)
    t2 = dict(t)
    t2["do_p"] = (t["do_p"].float() * 2).to(torch.bfloat16); t2["do_r"] = (t["do_r"].float() * 2).to(torch.bfloat16)
    got2, _ = pu.run_gpu(B, w, t2, flags=B.FLAG_ZERO_PROMPT_GRAD)
    for k in pu.GRADS:
        assert np.array_equal(got2[k], 2 * got[k]), k


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
    among them the first and last tokens, tokens either side of element offset 2^31, ends of branches, and
    prompt keys of one group (Eq. 2)."""
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
    _sample_rows(tb, f, out, rows, get=host)
    # response keys near the end of a branch (few rows see them): the last branch, one in the middle, the first
    cu_r = tb.cu_r
    a_k, a_v = pu.SampledError("dk_r"), pu.SampledError("dv_r")
    for b in (len(cu_r) - 2, (len(cu_r) - 1) // 2, 0):
        toks = [int(cu_r[b + 1]) - back for back in (9, 1) if int(cu_r[b + 1]) - back >= int(cu_r[b])]
        c = int(rng.integers(0, w.h_kv))
        dk, dv = ora.dkv_keys_block(tb, f["q_p"], f["k_p"], f["v_p"], f["do_p"], f["q_r"], f["k_r"], f["v_r"], f["do_r"], "r", toks, c)
        for i, tok in enumerate(toks):
            a_k.add(host(out["dk_r"][tok, c]), dk[i], (b, tok, c))
            a_v.add(host(out["dv_r"][tok, c]), dv[i], (b, tok, c))
    a_k.check(); a_v.check()
    # prompt keys (Eq. 2: summed over every branch and query head of the group, plus the later prompt rows):
    # tile-edge, middle and last keys of the group with the fewest response rows x keys, one KV head
    cost = [sum(bl) * (p + max(bl)) + p * p // 2 for p, bl in zip(w.prompt_len, w.branch_len)]
    g = int(np.argmin(cost))
    p0, P = int(tb.cu_p[g]), w.prompt_len[g]
    lo = max(0, P - 1024)   # keys of the last 1024 prompt tokens: the prefill's own (causal) part then stays small
    toks = sorted({p0 + lo, p0 + min(lo + 127, P - 1), p0 + min(lo + 128, P - 1), p0 + (lo + P) // 2, p0 + P - 1})
    c = int(rng.integers(0, w.h_kv))
    # one host copy of the group's slices (the block form reads them many times)
    b0, b1 = int(tb.cu_b[g]), int(tb.cu_b[g + 1])
    r0, r1 = int(tb.cu_r[b0]), int(tb.cu_r[b1])
    rep = w.h_q // w.h_kv
    sub_tb = ora.TreeBatch([P], [w.branch_len[g]], rep, 1, w.head_dim)
    hs = slice(c * rep, (c + 1) * rep)
    sub = {"q_p": t["q_p"][p0:p0 + P, hs], "k_p": t["k_p"][p0:p0 + P, c:c + 1], "v_p": t["v_p"][p0:p0 + P, c:c + 1],
           "do_p": t["do_p"][p0:p0 + P, hs], "q_r": t["q_r"][r0:r1, hs], "k_r": t["k_r"][r0:r1, c:c + 1],
           "v_r": t["v_r"][r0:r1, c:c + 1], "do_r": t["do_r"][r0:r1, hs]}
    sub = {k: v.float().cpu().numpy() for k, v in sub.items()}
    dk, dv = ora.dkv_keys_block(sub_tb, sub["q_p"], sub["k_p"], sub["v_p"], sub["do_p"], sub["q_r"], sub["k_r"], sub["v_r"],
                                sub["do_r"], "p", [tok - p0 for tok in toks], 0, block=512)
    a_k, a_v = pu.SampledError("dk_p"), pu.SampledError("dv_p")
    for i, tok in enumerate(toks):
        a_k.add(host(out["dk_p"][tok, c]), dk[i], (g, tok, c))
        a_v.add(host(out["dv_p"][tok, c]), dv[i], (g, tok, c))
    print(f"cfg{index} prompt keys of group {g}, KV head {c}: dk_p", a_k.check(), "dv_p", a_v.check())
    # every output finite (checked on the device)
    for k, v in out.items():
        if k != "ws":
            assert bool(torch.isfinite(v).all()), k
