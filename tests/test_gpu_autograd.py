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
    # the prompt-KV gradients as accumulated (fp32): the stated bounds, flat
    acc = {"dk_p": f64(plan.prompt_grad_fp32[0]), "dv_p": f64(plan.prompt_grad_fp32[1])}
    pu.assert_parity({**got, **acc}, {k: ref[k] for k in got})
    # ... and as autograd delivers them, in bf16 like their inputs: a value of magnitude 8-16 is rounded by up to
    # 3.1e-2 on delivery alone, so the element-wise bound is max(2e-2, six sigma of the modelled rounding error, delivery included)
    pu.assert_parity_elementwise(got, {k: ref[k] for k in got}, pu.rounding_error_sigma(w, t, bf16_prompt_grads=True))
    for k in ("dk_p", "dv_p"):   # the delivered copy is the accumulator rounded once
        assert np.array_equal(got[k], f64(torch.from_numpy(acc[k]).float().to(torch.bfloat16)))
