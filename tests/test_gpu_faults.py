"""Failure paths, exercised without faulting the GPU.

The faults are made by leaving work undone (the plan's test flags): a tile that is never loaded makes a
bounded device-side wait run out, and a lane table that has lost an item leaves that item's rows unwritten.
Checked: the call itself returns 0 (it only enqueues), the device status word names the wait that gave up,
the work accounting shows the shortfall, the outputs of the lane that gave up are untouched while the other
lanes' results are right, and the library keeps working afterwards.  Also: guard bands around every output
stay untouched on ragged and sharded workloads (no store past the end of a tensor or in front of it).
"""
import numpy as np
import pytest
import torch

from paper_2609_33133_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

# detail codes of the waits the two injected faults starve: the consumer's wait for the tile that never comes and the
# producer's wait for the ring slot that is therefore never released start within microseconds of each other, and
# whichever runs out first is recorded
FWD_STARVED, BWD_STARVED = (3, 4), (22, 23)     # WAIT_FWD_KV_FULL / _EMPTY, WAIT_BWD_QDO_FULL / _EMPTY
K_PREFILL_FWD, K_REPLAY_FWD, K_REPLAY_BWD = 0, 1, 2


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding
    return binding


W = wl.Workload("faults", [700, 200], [[300, 150], [260]], 4, 2, 128, 91)
LANES = 5


def _nan_outputs(B, plan):
    out = B.alloc_outputs(plan)
    for k, v in out.items():
        if k not in ("ws", "dk_p", "dv_p"):
            v.fill_(float("nan"))
    return out


def _lane_items(B, plan, base, width, lane):
    items = plan.metadata(base).reshape(-1, width)
    ptr, order = plan.metadata(base + 1), plan.metadata(base + 2)
    return [items[i] for i in order[ptr[lane]:ptr[lane + 1]]]


def test_forward_wait_runs_out_and_the_library_recovers(B):
    t_cpu = wl.make_tensors(W)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    ref = pu.run_oracle(W, t_cpu)
    plan = B.Plan(W.prompt_len, W.branch_len, W.h_q, W.h_kv, W.head_dim, device=0, n_lanes=LANES,
                  flags=B.FLAG_TEST_SHORT_WAIT | B.FLAG_TEST_SKIP_FWD_LOAD)
    out = _nan_outputs(B, plan)
    plan.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"])   # returns: it only enqueues
    torch.cuda.synchronize()                                                             # and the device comes back
    status, detail = plan.device_status()
    assert status == -5 and detail in FWD_STARVED, (status, detail)
    assert plan.device_status() == (0, 0)                      # the word is cleared by the read
    done, want = plan.items_completed(K_PREFILL_FWD)
    mine = _lane_items(B, plan, B.TBL_PREFILL_FWD_ITEMS, 12, 0)
    assert want - done == len(mine) > 0                        # lane 0 finished none of its items, the others all of theirs
    o, lse = out["o_p"].float().cpu().numpy(), out["lse_p"].cpu().numpy()
    untouched = np.zeros(o.shape[:2], dtype=bool)
    for it in mine:
        untouched[it[0]:it[0] + it[2], it[3]] = True
    assert np.isnan(o[untouched]).all() and np.isnan(lse.T[untouched]).all()
    got = np.where(untouched[:, :, None], ref["o_p"], o.astype(np.float64))   # every other row is right
    pu.assert_parity({"o_p": got, "lse_p": np.where(untouched.T, ref["lse_p"], lse.astype(np.float64))},
                     {"o_p": ref["o_p"], "lse_p": ref["lse_p"]})
    # a normal plan afterwards: the whole path matches the oracle
    got, plan2 = pu.run_gpu(B, W, t_cpu, n_lanes=LANES)
    pu.assert_parity_elementwise(got, ref, pu.rounding_error_sigma(W, t_cpu))
    for k in range(6):
        done, want = plan2.items_completed(k)
        assert done == want > 0, k


def test_backward_wait_runs_out_and_the_library_recovers(B):
    t_cpu = wl.make_tensors(W)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    good = B.Plan(W.prompt_len, W.branch_len, W.h_q, W.h_kv, W.head_dim, device=0, n_lanes=LANES)
    out = _nan_outputs(B, good)
    good.prefill_fwd(t["q_p"], t["k_p"], t["v_p"], out["o_p"], out["lse_p"], out["ws"])
    good.replay_fwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], out["ws"])
    bad = B.Plan(W.prompt_len, W.branch_len, W.h_q, W.h_kv, W.head_dim, device=0, n_lanes=LANES,
                 flags=B.FLAG_TEST_SHORT_WAIT | B.FLAG_TEST_SKIP_BWD_LOAD)
    bad.replay_bwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], t["do_r"],
                   out["dq_r"], out["dk_r"], out["dv_r"], out["dk_p"], out["dv_p"], out["ws"])
    torch.cuda.synchronize()
    status, detail = bad.device_status()
    assert status == -5 and detail in BWD_STARVED, (status, detail)
    done, want = bad.items_completed(K_REPLAY_BWD)
    mine = _lane_items(B, bad, B.TBL_REPLAY_BWD_ITEMS, 8, 0)
    assert want - done == len(mine) > 0
    dk = out["dk_r"].float().cpu().numpy()
    for it in mine:
        if it[4] == 0:                                         # a response-KV tile of the lane that gave up: never written
            assert np.isnan(dk[it[0]:it[0] + it[2], it[3]]).all()
    assert np.isfinite(out["dq_r"].float().cpu().numpy()).all()   # the query-side kernel ran after it, untroubled
    got, _ = pu.run_gpu(B, W, t_cpu, n_lanes=LANES)
    pu.assert_parity_elementwise(got, pu.run_oracle(W, t_cpu), pu.rounding_error_sigma(W, t_cpu))


def test_dropped_item_shows_in_the_work_accounting(B):
    t_cpu = wl.make_tensors(W)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    plan = B.Plan(W.prompt_len, W.branch_len, W.h_q, W.h_kv, W.head_dim, device=0, n_lanes=LANES, flags=B.FLAG_TEST_DROP_ITEM)
    out = _nan_outputs(B, plan)
    plan.replay_fwd(t["q_r"], t["k_r"], t["v_r"], t["k_p"], t["v_p"], out["o_r"], out["lse_r"], out["ws"])
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)                      # nothing timed out: the item was simply never run
    done, want = plan.items_completed(K_REPLAY_FWD)
    assert (done, want) == (want - 1, len(plan.metadata(B.TBL_REPLAY_FWD_ITEMS)) // 12)
    dropped = _lane_items(B, plan, B.TBL_REPLAY_FWD_ITEMS, 12, LANES - 1)[-1]
    o = out["o_r"].float().cpu().numpy()
    assert np.isnan(o[dropped[0]:dropped[0] + dropped[2], dropped[3]]).all()
    o[dropped[0]:dropped[0] + dropped[2], dropped[3]] = 0
    assert np.isfinite(o).all()


GUARD = 4096   # bytes of guard band on each side of every output


def _guarded(shape, dtype, fill):
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    pad = -n % 256
    raw = torch.full((GUARD + n + pad + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    view = raw[GUARD:GUARD + n].view(dtype).view(*shape)
    view.fill_(fill)
    return raw, view, n


@pytest.mark.parametrize("case", ["ragged", "sharded", "d64", "d96-sharded", "d40"])
def test_guard_bands_around_outputs_stay_untouched(B, case):
    w, splits = {
        "ragged": (wl.Workload("canary-ragged", [300, 1, 129], [[5, 130, 257], [1], [64, 200]], 4, 2, 128, 12), 0),
        "sharded": (wl.Workload("canary-sharded", [1100, 200], [[130, 64], [257]], 4, 2, 128, 21), 3),
        "d64": (wl.Workload("canary-d64", [77, 513], [[1, 129], [300]], 6, 2, 64, 13), 0),
        "d96-sharded": (wl.Workload("canary-d96", [600, 129], [[130, 257], [64]], 4, 2, 96, 14), 2),   # padded tiles
        "d40": (wl.Workload("canary-d40", [300], [[5, 130]], 4, 2, 40, 15), 0),
    }[case]
    t_cpu = wl.make_tensors(w)
    t = {k: v.cuda() for k, v in t_cpu.items()}
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0, kv_splits=splits)
    shapes = {k: (tuple(v.shape), v.dtype) for k, v in B.alloc_outputs(plan).items()}
    raws, out = {}, {}
    for k, (shape, dtype) in shapes.items():
        raws[k], out[k], _ = _guarded(shape, dtype, 0 if k in ("dk_p", "dv_p", "ws") else float("nan"))
    B.run_forward_backward(plan, t, out)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    for k, raw in raws.items():
        n = out[k].numel() * out[k].element_size()
        assert bool((raw[:GUARD] == 0xA5).all()), f"{k}: bytes in front of the tensor were written"
        assert bool((raw[GUARD + n:] == 0xA5).all()), f"{k}: bytes past the end of the tensor were written"
    got = {k: v.float().cpu().numpy().astype(np.float64) for k, v in out.items() if k != "ws"}
    pu.assert_parity_elementwise(got, pu.run_oracle(w, t_cpu), pu.rounding_error_sigma(w, t_cpu))
