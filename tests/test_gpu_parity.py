"""GPU parity: the CUDA path, called through the C interface, against the fp64 oracle, element by element."""
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


def _wl(name, pl, bl, hq, hkv, d, seed):
    return wl.Workload(name, pl, bl, hq, hkv, d, seed)


SMALL = [
    _wl("cfg1", [256], [[128] * 4], 4, 4, 64, 1001),
    _wl("d128-gqa", [384], [[256, 128]], 4, 2, 128, 11),
    _wl("ragged", [300, 1, 129], [[5, 130, 257], [1], [64, 200]], 4, 2, 128, 12),
    _wl("ragged-d64", [77, 513], [[1, 129], [300]], 6, 2, 64, 13),
    _wl("prompt-only", [200, 130], [[], []], 2, 1, 128, 14),
    _wl("tiny", [1], [[1]], 1, 1, 64, 15),
    _wl("g7", [640], [[192] * 3], 14, 2, 128, 16),
    _wl("d64-multi", [900, 260], [[700, 300, 129], [515]], 8, 2, 64, 17),   # head dim 64 over many tiles, GQA 4:1
]


@pytest.mark.parametrize("w", SMALL, ids=[w.name for w in SMALL])
def test_small_cases_match_oracle(B, w):
    t = wl.make_tensors(w)
    got, _ = pu.run_gpu(B, w, t)
    if w.name == "tiny":
        # One query row over two keys, 64 numbers per tensor: the relative-L2 figure is a statistic over a
        # tensor and does not average here (bf16 rounding of O, P and dS is 2^-9 per element and the two-key
        # softmax backward cancels).  Measured 1.3e-2; bound for this case only 3e-2.  The absolute bounds stay.
        wide = {k: {"rel_l2": 3e-2} for k in ("o_p", "o_r", *pu.GRADS)}
        pu.assert_parity(got, pu.run_oracle(w, t), exceptions=wide)
        return
    pu.assert_parity(got, pu.run_oracle(w, t))


@pytest.mark.parametrize("splits", [2, 3, 8])
def test_split_prompt_kv_matches_oracle(B, splits):
    w = _wl("split", [1100, 200], [[130, 64], [257]], 4, 2, 128, 21)
    t = wl.make_tensors(w)
    got, plan = pu.run_gpu(B, w, t, kv_splits=splits)
    assert plan.metadata(B.TBL_GROUP_SPLITS).max() > 1
    pu.assert_parity(got, pu.run_oracle(w, t))


def test_split_prompt_kv_head_dim_64(B):
    w = _wl("split-d64", [1300], [[200, 333]], 4, 1, 64, 22)
    t = wl.make_tensors(w)
    got, plan = pu.run_gpu(B, w, t, kv_splits=4)
    assert plan.metadata(B.TBL_GROUP_SPLITS).max() > 1
    pu.assert_parity(got, pu.run_oracle(w, t))


def test_few_lanes_and_zero_flag(B):
    """Many items per lane (barrier phases wrap many times) and the accumulator-clearing flag."""
    w = _wl("lanes", [700], [[300, 150, 420]], 4, 2, 128, 31)
    t = wl.make_tensors(w)
    ref = pu.run_oracle(w, t)
    got, _ = pu.run_gpu(B, w, t, n_lanes=3, flags=B.FLAG_ZERO_PROMPT_GRAD)
    pu.assert_parity(got, ref)


def test_results_are_bitwise_repeatable(B):
    """No atomics anywhere: every tile has one owner and a fixed summation order, so all outputs,
    the many-to-one prompt-KV gradients of Eq. 2 included, are bitwise equal across runs."""
    w = _wl("det", [512], [[256] * 4], 8, 2, 128, 41)
    t = wl.make_tensors(w)
    a, _ = pu.run_gpu(B, w, t)
    b, _ = pu.run_gpu(B, w, t)
    for k in a:
        assert np.array_equal(a[k], b[k]), k


def test_flattened_baseline_matches_tree(B):
    """The no-reuse baseline (same kernels, prompt duplicated per branch) gives the tree's results;
    its per-copy prompt gradients add up to the tree's (Eq. 2)."""
    w = _wl("flat", [260], [[100, 190]], 4, 2, 128, 51)
    t = wl.make_tensors(w)
    ref = pu.run_oracle(w, t)
    fw, ft = w.flattened(), wl.flatten_tensors(w, t)
    empty = lambda h: torch.empty((0, h, w.head_dim), dtype=torch.bfloat16)
    ft.update({"q_r": empty(w.h_q), "k_r": empty(w.h_kv), "v_r": empty(w.h_kv), "do_r": empty(w.h_q)})
    got, _ = pu.run_gpu(B, fw, ft)
    P, off = 260, 0
    dk = np.zeros_like(ref["dk_p"]); dv = np.zeros_like(ref["dv_p"]); dq = np.zeros_like(ref["dq_p"])
    r_off = 0
    for r in (100, 190):
        dk += got["dk_p"][off:off + P]; dv += got["dv_p"][off:off + P]; dq += got["dq_p"][off:off + P]
        sl = slice(off + P, off + P + r)
        part = {"o_r": got["o_p"][sl], "dq_r": got["dq_p"][sl], "dk_r": got["dk_p"][sl], "dv_r": got["dv_p"][sl]}
        refp = {k: ref[k][r_off:r_off + r] for k in part}
        pu.assert_parity(part, refp)
        np.testing.assert_allclose(got["lse_p"][:, sl], ref["lse_r"][:, r_off:r_off + r], atol=pu.LSE_ABS)
        off += P + r; r_off += r
    pu.assert_parity({"dk_p": dk, "dv_p": dv, "dq_p": dq}, {k: ref[k] for k in ("dk_p", "dv_p", "dq_p")})


def test_cuda_graph_replay_is_bitwise_the_eager_step(B):
    """The four entry points capture into a CUDA graph (no allocation or synchronisation in the launch path)."""
    w = _wl("graph", [256], [[128] * 4], 4, 4, 64, 61)
    t = {k: v.cuda() for k, v in wl.make_tensors(w).items()}
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0, flags=B.FLAG_ZERO_PROMPT_GRAD)
    out = B.alloc_outputs(plan)
    B.run_forward_backward(plan, t, out)
    torch.cuda.synchronize()
    eager = {k: v.clone() for k, v in out.items() if k != "ws"}
    g = B.capture_step(plan, t, out)
    for k, v in out.items():
        if k not in ("ws", "dk_p", "dv_p"):
            v.fill_(float("nan"))
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    for k, v in eager.items():
        assert torch.equal(v, out[k]), k
