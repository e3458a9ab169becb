"""augtree_replay_fwd_static: the sharded replay forward for callers that cannot allocate scratch.

Some users of this library run where device allocation is not theirs to do (a plug-in handed
pre-existing tensors by a runtime that owns the allocator, a loop that must never touch the allocator).
They cannot supply the workspace the sharded forward needs, so this entry point keeps that scratch in a
32 MiB array inside the library's device image.  The test calls it through the C interface twice in a row
and checks each result against the ordinary entry point (which gets a torch-allocated workspace) with the
tolerances of the other parity tests; the two paths run the same kernels, so they also agree bit for bit.
Each result is also compared with the fp64 oracle directly.  It also checks that free device memory does not move across a call and that an oversized plan is refused.
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


def _forward(B, plan, t, static):
    hq, d = plan.h_q, plan.head_dim
    o = torch.full((plan.total_r, hq, d), float("nan"), device="cuda", dtype=torch.bfloat16)
    lse = torch.full((hq, plan.total_r), float("nan"), device="cuda", dtype=torch.float32)
    if static:
        plan.replay_fwd_static(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], o, lse)
    else:
        ws = torch.empty(max(plan.ws_fwd_bytes, 256), device="cuda", dtype=torch.uint8)
        plan.replay_fwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], o, lse, ws)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def test_static_scratch_matches_workspace_variant_twice(B):
    for seed, pl, bl in [(61, [1100, 300], [[130, 64], [257]]), (62, [700], [[200, 90, 33]])]:   # two calls, different shapes
        w = wl.Workload("noalloc", pl, bl, 4, 2, 128, seed)
        t = {k: v.cuda() for k, v in wl.make_tensors(w).items()}
        plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0, kv_splits=3)
        assert 0 < plan.ws_fwd_bytes <= B.STATIC_SCRATCH_BYTES
        ref_o, ref_lse = _forward(B, plan, t, static=False)
        got_o, got_lse = _forward(B, plan, t, static=True)       # first call on the device also does the set-up
        o = torch.empty((plan.total_r, 4, 128), device="cuda", dtype=torch.bfloat16)
        lse = torch.empty((4, plan.total_r), device="cuda", dtype=torch.float32)
        free1 = torch.cuda.mem_get_info()[0]
        plan.replay_fwd_static(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], o, lse)   # second call in a row
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free1, "the call changed the amount of free device memory"
        got_o2, got_lse2 = o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
        oracle = pu.run_oracle(w, wl.make_tensors(w))
        oracle = {"o_r": oracle["o_r"], "lse_r": oracle["lse_r"]}
        for go, gl in ((got_o, got_lse), (got_o2, got_lse2)):
            rows = pu.errors({"o_r": go, "lse_r": gl}, {"o_r": ref_o, "lse_r": ref_lse})
            assert rows["o_r"][0] <= pu.REL_L2 and rows["o_r"][1] <= pu.MAX_ABS and rows["lse_r"][1] <= pu.LSE_ABS, rows
            assert np.array_equal(go, ref_o) and np.array_equal(gl, ref_lse)
            pu.assert_parity({"o_r": go, "lse_r": gl}, oracle)


def test_static_scratch_refuses_oversized_plan(B):
    # 8 shards x 20000 response tokens x 8 heads x 129 floats = 660 MB of partials: over the 32 MiB array
    plan = B.Plan([4096], [[20000]], 8, 2, 128, device=0, kv_splits=8)
    assert plan.ws_fwd_bytes > B.STATIC_SCRATCH_BYTES
    x = torch.empty(16, device="cuda", dtype=torch.bfloat16)
    f = torch.empty(16, device="cuda", dtype=torch.float32)
    with pytest.raises(B.AugtreeError) as e:
        plan.replay_fwd_static(x, x, x, x, x, x, f)
    assert e.value.code == -3
