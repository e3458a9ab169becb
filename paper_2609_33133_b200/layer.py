"""One decoder layer and the language-model loss on a prompt-sharing tree (integration around the attention path).

What the method changes in a model is its self-attention operator and nothing else: loss, gradient synchronisation
and optimizer stay the base trainer's (Sec. 4, attention dispatch).  This module is that seam written out for a
standard pre-norm decoder layer:

* the prompt of a group is embedded and pushed through the layer ONCE, its responses once each, never the G flattened
  copies (Sec. 3.2, prefill once / replay);
* positions: prompt token i sits at position i, token t of a response at P_g + t, as in its flattened sequence, so
  RoPE gives every branch the keys and queries it would have had on its own;
* attention: `autograd.tree_attention` (the C-ABI path; everything else here is plain torch: library GEMMs,
  element-wise ops);
* loss: token-level cross-entropy on the response tokens.  The first token of every response is scored from the
  LAST PROMPT hidden state of its group, and that loss flows back through the prompt's own graph (Sec. 3.2, response
  replay): that state therefore carries one target per branch.

Nothing here is on the measured hot path; tests compare loss and weight gradients with the flattened execution.
"""
from __future__ import annotations

import torch
import torch.nn.functional as F

from . import binding as B
from .autograd import tree_attention

BF16 = torch.bfloat16


def tree_positions(plan: B.Plan, device="cuda"):
    """Position ids of the packed prompt tokens and of the packed response tokens."""
    pos_p = torch.cat([torch.arange(P, device=device) for P in plan.prompt_len]) if plan.total_p else torch.zeros(0, device=device)
    pos_r = [torch.arange(P, P + r, device=device) for P, rs in zip(plan.prompt_len, plan.branch_len) for r in rs]
    pos_r = torch.cat(pos_r) if pos_r else torch.zeros(0, dtype=torch.long, device=device)
    return pos_p.long(), pos_r.long()


def seam_index(plan: B.Plan, device="cuda"):
    """For every packed response token, where the hidden state that predicts it lives: (from_prompt mask, index).
    The first token of a response is predicted by the last prompt token of its group, every other token by the
    response token before it."""
    from_prompt, index = [], []
    p0 = r0 = 0
    for P, rs in zip(plan.prompt_len, plan.branch_len):
        for r in rs:
            from_prompt += [True] + [False] * (r - 1)
            index += [p0 + P - 1] + list(range(r0, r0 + r - 1))
            r0 += r
        p0 += P
    return torch.tensor(from_prompt, dtype=torch.bool, device=device), torch.tensor(index, dtype=torch.long, device=device)


def rope(x, pos, theta=10000.0):
    """Rotary position embedding, rotate-half convention; x [tokens, heads, d] (any float dtype), pos [tokens]."""
    d = x.shape[-1]
    inv = theta ** (-torch.arange(0, d, 2, device=x.device, dtype=torch.float32) / d)
    ang = pos.to(torch.float32)[:, None] * inv[None, :]
    cos, sin = ang.cos()[:, None, :], ang.sin()[:, None, :]
    x1, x2 = x.float()[..., : d // 2], x.float()[..., d // 2:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1).to(x.dtype)


def rms_norm(x, weight, eps=1e-6):
    x = x.float()
    return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + eps) * weight


class TreeDecoderLayer(torch.nn.Module):
    """Pre-norm decoder layer: RMSNorm, GQA self-attention with RoPE, SwiGLU MLP.  fp32 parameters and residual
    stream, bf16 GEMMs and attention."""

    def __init__(self, hidden, h_q, h_kv, head_dim, mlp_hidden, rope_theta=10000.0):
        super().__init__()
        self.h_q, self.h_kv, self.head_dim, self.rope_theta = h_q, h_kv, head_dim, rope_theta
        mk = lambda o, i: torch.nn.Parameter(torch.randn(o, i) * i ** -0.5)
        self.wq, self.wk, self.wv = mk(h_q * head_dim, hidden), mk(h_kv * head_dim, hidden), mk(h_kv * head_dim, hidden)
        self.wo = mk(hidden, h_q * head_dim)
        self.w_gate, self.w_up, self.w_down = mk(mlp_hidden, hidden), mk(mlp_hidden, hidden), mk(hidden, mlp_hidden)
        self.norm1, self.norm2 = torch.nn.Parameter(torch.ones(hidden)), torch.nn.Parameter(torch.ones(hidden))

    @staticmethod
    def _lin(x, w):
        return F.linear(x.to(BF16), w.to(BF16))

    def qkv(self, x, pos):
        """Projections of the normalised stream with RoPE on q and k: bf16 [tokens, heads, d], contiguous."""
        h = rms_norm(x, self.norm1)
        t = x.shape[0]
        q = rope(self._lin(h, self.wq).view(t, self.h_q, self.head_dim), pos, self.rope_theta)
        k = rope(self._lin(h, self.wk).view(t, self.h_kv, self.head_dim), pos, self.rope_theta)
        v = self._lin(h, self.wv).view(t, self.h_kv, self.head_dim)
        return q.contiguous(), k.contiguous(), v.contiguous()

    def after_attention(self, x, o):
        """Output projection, residual, MLP, residual."""
        x = x + self._lin(o.reshape(o.shape[0], -1), self.wo).float()
        h = rms_norm(x, self.norm2)
        return x + self._lin(F.silu(self._lin(h, self.w_gate).float()) * self._lin(h, self.w_up).float(), self.w_down).float()

    def forward(self, plan: B.Plan, x_p, x_r, pos_p, pos_r):
        """x_p [sumP, hidden], x_r [sumR, hidden] fp32 -> the same shapes; the prompt is computed once per group."""
        q_p, k_p, v_p = self.qkv(x_p, pos_p)
        q_r, k_r, v_r = self.qkv(x_r, pos_r)
        o_p, o_r = tree_attention(plan, q_p, k_p, v_p, q_r, k_r, v_r)
        return self.after_attention(x_p, o_p), self.after_attention(x_r, o_r)


def tree_lm_loss(plan: B.Plan, h_p, h_r, lm_head, resp_tokens, seam=None):
    """Sum of the token-level cross-entropies of all response tokens.  h_p, h_r: final hidden states of the packed prompt
    and response tokens; lm_head [vocab, hidden]; resp_tokens [sumR] the packed response token ids."""
    from_prompt, index = seam if seam is not None else seam_index(plan, h_p.device)
    src = torch.where(from_prompt[:, None], h_p[index.clamp(max=max(h_p.shape[0] - 1, 0))], h_r[index.clamp(max=max(h_r.shape[0] - 1, 0))])
    logits = F.linear(src.to(BF16), lm_head.to(BF16)).float()
    return F.cross_entropy(logits, resp_tokens, reduction="sum")
