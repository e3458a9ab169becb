"""torch.autograd wrapper around the four entry points (argument marshalling only).

`tree_attention(plan, q_p, k_p, v_p, q_r, k_r, v_r)` returns `(o_p, o_r)` for the packed prompt and
response tokens of a plan's groups; backward fills the gradients of all six inputs.  The order inside
backward is the one the method requires (Sec. 3.2): the replay backward first, which seeds the shared
prompt-KV gradient with the sum over every branch (Eq. 2), then the prefill backward, which adds the
prompt's own contribution and pushes the total through the prefill pass.  Inputs and outputs are bf16
`[tokens, heads, head_dim]`; the prompt-KV gradients are accumulated in fp32 and cast once at the end
(autograd hands a gradient back in its input's dtype).  The fp32 accumulators of the latest backward stay
available as `plan.prompt_grad_fp32 = (dK_P, dV_P)` for callers that want them unrounded.
"""
from __future__ import annotations

import torch

from . import binding as B


class _TreeAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan, q_p, k_p, v_p, q_r, k_r, v_r):
        for t in (q_p, k_p, v_p, q_r, k_r, v_r):
            if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
                raise ValueError("tree_attention takes contiguous bf16 CUDA tensors")
        dev = q_p.device
        hq, d = plan.h_q, plan.head_dim
        o_p = torch.empty((plan.total_p, hq, d), device=dev, dtype=torch.bfloat16)
        o_r = torch.empty((plan.total_r, hq, d), device=dev, dtype=torch.bfloat16)
        lse_p = torch.empty((hq, plan.total_p), device=dev, dtype=torch.float32)
        lse_r = torch.empty((hq, plan.total_r), device=dev, dtype=torch.float32)
        ws = torch.empty(max(plan.ws_fwd_bytes, plan.ws_bwd_bytes, 256), device=dev, dtype=torch.uint8)
        plan.prefill_fwd(q_p, k_p, v_p, o_p, lse_p, ws)
        plan.replay_fwd(q_r, k_r, v_r, k_p, v_p, o_r, lse_r, ws)
        ctx.plan, ctx.ws = plan, ws
        ctx.save_for_backward(q_p, k_p, v_p, q_r, k_r, v_r, o_p, lse_p, o_r, lse_r)
        return o_p, o_r

    @staticmethod
    def backward(ctx, do_p, do_r):
        plan, ws = ctx.plan, ctx.ws
        q_p, k_p, v_p, q_r, k_r, v_r, o_p, lse_p, o_r, lse_r = ctx.saved_tensors
        dev = q_p.device
        hq, hkv, d = plan.h_q, plan.h_kv, plan.head_dim
        bf = torch.bfloat16
        do_p = torch.zeros_like(o_p) if do_p is None else do_p.to(bf).contiguous()
        do_r = torch.zeros_like(o_r) if do_r is None else do_r.to(bf).contiguous()
        dq_p = torch.empty((plan.total_p, hq, d), device=dev, dtype=bf)
        dq_r = torch.empty((plan.total_r, hq, d), device=dev, dtype=bf)
        dk_r = torch.empty((plan.total_r, hkv, d), device=dev, dtype=bf)
        dv_r = torch.empty((plan.total_r, hkv, d), device=dev, dtype=bf)
        dk_acc = torch.zeros((plan.total_p, hkv, d), device=dev, dtype=torch.float32)
        dv_acc = torch.zeros((plan.total_p, hkv, d), device=dev, dtype=torch.float32)
        dk_p = torch.empty((plan.total_p, hkv, d), device=dev, dtype=bf)
        dv_p = torch.empty((plan.total_p, hkv, d), device=dev, dtype=bf)
        plan.replay_bwd(q_r, k_r, v_r, k_p, v_p, o_r, lse_r, do_r, dq_r, dk_r, dv_r, dk_acc, dv_acc, ws)
        plan.prefill_bwd(q_p, k_p, v_p, o_p, lse_p, do_p, dk_acc, dv_acc, dq_p, dk_p, dv_p, ws)
        plan.prompt_grad_fp32 = (dk_acc, dv_acc)
        return None, dq_p, dk_p, dv_p, dq_r, dk_r, dv_r


def tree_attention(plan: B.Plan, q_p, k_p, v_p, q_r, k_r, v_r):
    """Prompt-sharing tree attention of a plan's groups; differentiable in all six tensors."""
    return _TreeAttention.apply(plan, q_p, k_p, v_p, q_r, k_r, v_r)
