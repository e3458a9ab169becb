"""MoveQ (Sec. 3.3) emulated on one GPU: n ranks' prompt-KV shards stay put, every rank computes every response
query's partial state over its shard through the library's partial-state entry points, the states are merged, and
the backward pass sums the ranks' dQ contributions while each shard's dK_P / dV_P stays local (Eq. 2).  All ranks
run one after the other in one process, so nothing here waits on another rank.  Compared with the fp64 oracle.
"""
import numpy as np
import pytest
import torch

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


CASES = {
    "two-groups": wl.Workload("moveq-a", [700, 300], [[300, 150, 420], [257]], 4, 2, 128, 81),
    "gqa7-d128": wl.Workload("moveq-b", [1100], [[130, 64, 200, 90, 333]], 14, 2, 128, 82),
    "d64": wl.Workload("moveq-c", [513, 260], [[129, 1], [300, 77]], 8, 2, 64, 83),
    "d96": wl.Workload("moveq-d", [640], [[200, 130, 65]], 8, 2, 96, 85),     # head dimension padded to the 128-wide tile
}


@pytest.mark.parametrize("world", [2, 3, 4])
@pytest.mark.parametrize("case", list(CASES))
def test_moveq_emulation_matches_oracle(B, case, world):
    from paper_2609_33133_b200 import cp
    w = CASES[case]
    t_cpu = wl.make_tensors(w)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    res = cp.moveq_emulate(B, w, t, world)
    # the prompt's own pass (not sharded here): prefill forward, then its backward ADDS to the MoveQ seeds
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0)
    out = B.alloc_outputs(plan)
    out["dk_p"].copy_(res["dk_p"]); out["dv_p"].copy_(res["dv_p"])
    plan.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"])
    plan.prefill_bwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], t["do_p"], out["dk_p"], out["dv_p"], out["dq_p"], None, None, out["ws"])
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    f64 = lambda x: x.float().cpu().numpy().astype(np.float64)
    got = {k: f64(res[k]) for k in ("o_r", "lse_r", "dq_r", "dk_r", "dv_r")}
    got.update({k: f64(out[k]) for k in ("o_p", "lse_p", "dq_p", "dk_p", "dv_p")})
    ref = pu.run_oracle(w, t_cpu)
    pu.assert_parity_elementwise(got, ref, pu.rounding_error_sigma(w, t_cpu))
    # one rank is the unsharded replay: the same kernels, so the merged result is the library's own bit for bit
    if world == 2:
        whole, _ = pu.run_gpu(B, w, t_cpu)
        one = cp.moveq_emulate(B, w, t, 1)
        assert np.array_equal(f64(one["lse_r"]), whole["lse_r"])
        assert np.abs(f64(one["o_r"]) - whole["o_r"]).max() <= 2.0 ** -7 * np.abs(whole["o_r"]).max()   # fp32 state -> bf16 once more


@pytest.mark.parametrize("s_lanes,d_lane,rounds", [(1, 2, 1), (2, 2, 1), (2, 3, 2), (4, 1, 1)])
def test_treemovekv_emulation_matches_oracle(B, s_lanes, d_lane, rounds):
    """TreeMoveKV: lanes from the replay-grid placement (Eq. 6), prompt-KV shards going round each lane's ring, the
    shards' gradient accumulators going round again; every path stays on one rank."""
    from paper_2609_33133_b200 import cp
    w = wl.Workload("tmkv", [900], [[300, 150, 420, 64, 257, 130]], 8, 2, 128, 84)
    t_cpu = wl.make_tensors(w)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    res = cp.treemovekv_emulate(B, w, t, s_lanes, d_lane, rounds)
    x_round, x_lane = res.pop("placement")
    assert max(x_round) < rounds and max(x_lane) < s_lanes and len(x_lane) == 6
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0)
    out = B.alloc_outputs(plan)
    out["dk_p"].copy_(res["dk_p"]); out["dv_p"].copy_(res["dv_p"])
    plan.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"])
    plan.prefill_bwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], t["do_p"], out["dk_p"], out["dv_p"], out["dq_p"], None, None, out["ws"])
    torch.cuda.synchronize()
    f64 = lambda x: x.float().cpu().numpy().astype(np.float64)
    got = {k: f64(res[k]) for k in ("o_r", "lse_r", "dq_r", "dk_r", "dv_r")}
    got.update({k: f64(out[k]) for k in ("o_p", "lse_p", "dq_p", "dk_p", "dv_p")})
    pu.assert_parity_elementwise(got, pu.run_oracle(w, t_cpu), pu.rounding_error_sigma(w, t_cpu))
