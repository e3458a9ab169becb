"""The torch.autograd wrapper: gradients of all six inputs through loss.backward() against the oracle."""
import numpy as np
import pytest
import torch

from paper_2609_33133_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def test_autograd_wrapper_matches_oracle():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding as B
    from paper_2609_33133_b200.autograd import tree_attention
    w = wl.Workload("autograd", [300, 129], [[130, 64, 257], [200]], 8, 2, 128, 77)
    t = wl.make_tensors(w)   # seeds as generated: N(0, 1), unscaled
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=0)
    x = {k: t[k].cuda().requires_grad_(True) for k in ("q_p", "k_p", "v_p", "q_r", "k_r", "v_r")}
    o_p, o_r = tree_attention(plan, x["q_p"], x["k_p"], x["v_p"], x["q_r"], x["k_r"], x["v_r"])
    # L = <O_P, dO_P> + <O_R, dO_R>: its gradient with respect to the outputs is the seeded dO
    loss = (o_p.float() * t["do_p"].cuda().float()).sum() + (o_r.float() * t["do_r"].cuda().float()).sum()
    loss.backward()
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    ref = pu.run_oracle(w, t)
    f64 = lambda v: v.detach().float().cpu().numpy().astype(np.float64)
    got = {"o_p": f64(o_p), "o_r": f64(o_r), "dq_p": f64(x["q_p"].grad), "dk_p": f64(x["k_p"].grad), "dv_p": f64(x["v_p"].grad),
           "dq_r": f64(x["q_r"].grad), "dk_r": f64(x["k_r"].grad), "dv_r": f64(x["v_r"].grad)}
    ref = {k: ref[k] for k in got}
    sigma = pu.rounding_error_sigma(w, t, bf16_prompt_grads=True)
    # as autograd delivers them (every gradient in bf16, like its input): relative L2 as stated; element-wise
    # max(2e-2, six sigma of the modelled rounding error, delivery included), because a bf16 value of magnitude
    # 4-8 is rounded by up to 1.6e-2 on delivery alone and the first rows of a prompt carry large dS roundings
    # (measured here: one element of dq_p, |ref| = 6.6, off by 2.4e-2)
    pu.assert_parity_elementwise(got, ref, sigma)
    # the outputs and the prompt-KV gradients as accumulated (fp32): the stated bounds, flat
    acc = {"dk_p": f64(plan.prompt_grad_fp32[0]), "dv_p": f64(plan.prompt_grad_fp32[1])}
    flat = ("o_p", "o_r", "dk_p", "dv_p")
    pu.assert_parity({**{k: got[k] for k in ("o_p", "o_r")}, **acc}, {k: ref[k] for k in flat})
    for k in ("dk_p", "dv_p"):   # the delivered copy is the accumulator rounded once
        assert np.array_equal(got[k], f64(torch.from_numpy(acc[k]).float().to(torch.bfloat16)))
