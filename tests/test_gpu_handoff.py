"""The two backward paths: recomputing (seven GEMMs per tile pair) and dS hand-off (five).  The key-side kernel is the
same code in both, so dK, dV and the prompt accumulators must agree bit for bit; dQ comes from the key-side kernel's
stored dS on one path and from the query-side kernel's own recomputation on the other, so it is compared with the oracle
on both paths."""
import numpy as np
import pytest
import torch

from paper_2609_33133_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding
    return binding


CASES = [
    ("one-group-d128", [700], [[300, 150, 420]], 8, 2, 128, 0),
    ("ragged-d64", [129, 1000], [[1, 257], [640, 64, 130, 127]], 4, 4, 64, 0),
    ("gqa7-d128", [1024], [[256] * 4], 14, 2, 128, 0),
    ("sharded-prompt", [2048], [[384, 200]], 8, 4, 128, 4),
    ("no-branches", [300, 513], [[], []], 4, 2, 64, 0),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_handoff_and_recompute_paths_agree(B, case):
    name, pl, bl, hq, hkv, d, splits = case
    w = wl.Workload(name, pl, bl, hq, hkv, d, seed=77)
    t = wl.make_tensors(w, device="cpu")
    ref = pu.run_oracle(w, t)
    re_, plan = pu.run_gpu(B, w, t, kv_splits=splits, handoff_limit=0)
    ho_, plan2 = pu.run_gpu(B, w, t, kv_splits=splits, handoff_limit=1 << 40)
    assert plan2.workspace_bytes(1 << 40) >= plan2.ws_bwd_handoff_bytes > plan2.ws_bwd_bytes
    assert plan.workspace_bytes(0) < plan.ws_bwd_handoff_bytes
    for k in ("o_p", "lse_p", "o_r", "lse_r", "dk_r", "dv_r", "dk_p", "dv_p"):
        assert np.array_equal(re_[k], ho_[k]), k
    pu.assert_parity(re_, ref)
    pu.assert_parity(ho_, ref)
    # every item of every schedule ran on both paths
    for p in (plan, plan2):
        for kind in range(6):
            done, want = p.items_completed(kind)
            assert done == want, (kind, done, want)


def test_partial_state_backward_takes_the_handoff_too(B):
    """replay_bwd_state (prompt keys only, fp32 dQ contribution) with and without the hand-off scratch."""
    w = wl.Workload("cp-shard", [640], [[200, 330]], 8, 2, 128, seed=5)
    t = {k: v.cuda() for k, v in wl.make_tensors(w, device="cpu").items()}
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0)
    out = B.alloc_outputs(plan, handoff_limit=1 << 40)
    B.run_forward_backward(plan, t, out)
    res = []
    for nbytes in (plan.ws_bwd_bytes, plan.ws_bwd_handoff_bytes):
        ws = torch.empty(max(nbytes, 256), device="cuda", dtype=torch.uint8)
        dq = torch.full((plan.total_r, w.h_q, w.head_dim), float("nan"), device="cuda", dtype=torch.float32)
        dk = torch.zeros((plan.total_p, w.h_kv, w.head_dim), device="cuda", dtype=torch.float32)
        dv = torch.zeros_like(dk)
        for include_own in (0, 1):
            plan.replay_bwd_state(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], t["do_r"], dq,
                                  out["dk_r"], out["dv_r"], dk, dv, include_own, ws)
            torch.cuda.synchronize()
            assert plan.device_status() == (0, 0)
            res.append((include_own, dq.clone(), dk.clone(), dv.clone()))
    for (a, dq_a, dk_a, dv_a), (b, dq_b, dk_b, dv_b) in zip(res[:2], res[2:]):
        assert a == b
        assert torch.equal(dk_a, dk_b) and torch.equal(dv_a, dv_b)
        err = (dq_a - dq_b).abs().max().item()
        assert err <= 1e-3 * max(1.0, dq_a.abs().max().item()), err   # fp32 sums over dS values that differ by a bf16 step here and there


def test_workspace_aligned_to_16_bytes_only_takes_the_recomputing_path(B):
    """The hand-off tiles are written with 32-byte stores; a scratch block that is large enough but only 16-byte aligned
    must not take that path: its dQ is then bit for bit the recomputing kernel's."""
    w = wl.Workload("align", [400], [[150, 260]], 4, 2, 128, seed=9)
    t = {k: v.cuda() for k, v in wl.make_tensors(w, device="cpu").items()}
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0)
    out = B.alloc_outputs(plan, handoff_limit=0)
    B.run_forward_backward(plan, t, out)
    torch.cuda.synchronize()
    want = {k: out[k].clone() for k in ("dq_r", "dk_r", "dv_r", "dk_p", "dv_p")}
    big = torch.empty(plan.ws_bwd_handoff_bytes + 64, device="cuda", dtype=torch.uint8)
    off = (-big.data_ptr()) % 32 + 16                     # 16 modulo 32
    ws = big[off:off + plan.ws_bwd_handoff_bytes]
    assert ws.data_ptr() % 32 == 16 and ws.numel() >= plan.ws_bwd_handoff_bytes
    out["dk_p"].zero_(); out["dv_p"].zero_()
    for k in ("dq_r", "dk_r", "dv_r"):
        out[k].fill_(float("nan"))
    plan.replay_bwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], t["do_r"],
                    out["dq_r"], out["dk_r"], out["dv_r"], out["dk_p"], out["dv_p"], ws)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    # dk_p / dv_p of the reference run also hold the prefill call's share: compare the replay outputs only
    for k in ("dq_r", "dk_r", "dv_r"):
        assert torch.equal(out[k], want[k]), k
