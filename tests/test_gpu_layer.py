"""Model-level check of the seam around the attention path: a two-layer decoder with a language-model head, trained on a
prompt-sharing tree (prompt once, responses replayed, first response token scored from the last prompt state) against
the same model on the flattened sequences (every branch as its own prompt + response sequence, plain causal
attention in torch).  Loss and weight gradients must agree, and so must the loss trajectory over a few optimizer
steps: the check the paper reports for its engine (equal loss trajectories on identical replay inputs, Sec. 5,
correctness)."""
import copy

import pytest
import torch
import torch.nn.functional as F

pytestmark = pytest.mark.gpu

HIDDEN, H_Q, H_KV, MLP, VOCAB, LAYERS = 256, 4, 2, 512, 503, 2


@pytest.fixture(scope="module")
def mods():
    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding, layer
    return binding, layer


class TinyLM(torch.nn.Module):
    def __init__(self, L, D):
        super().__init__()
        self.emb = torch.nn.Parameter(torch.randn(VOCAB, HIDDEN) * 0.5)
        self.layers = torch.nn.ModuleList([L.TreeDecoderLayer(HIDDEN, H_Q, H_KV, D, MLP) for _ in range(LAYERS)])
        self.norm = torch.nn.Parameter(torch.ones(HIDDEN))
        self.head = torch.nn.Parameter(torch.randn(VOCAB, HIDDEN) * HIDDEN ** -0.5)


def tree_loss(L, model, plan, prompt_tok, resp_tok):
    pos_p, pos_r = L.tree_positions(plan)
    x_p, x_r = model.emb[prompt_tok], model.emb[resp_tok]
    for layer in model.layers:
        x_p, x_r = layer(plan, x_p, x_r, pos_p, pos_r)
    return L.tree_lm_loss(plan, L.rms_norm(x_p, model.norm), L.rms_norm(x_r, model.norm), model.head, resp_tok)


def causal_attention_reference(q, k, v):
    """Plain causal GQA attention of one sequence in fp32 on the bf16 inputs; bf16 output like the kernels'."""
    rep = q.shape[1] // k.shape[1]
    qf, kf, vf = q.float().transpose(0, 1), k.float().repeat_interleave(rep, 1).transpose(0, 1), v.float().repeat_interleave(rep, 1).transpose(0, 1)
    o = F.scaled_dot_product_attention(qf[None], kf[None], vf[None], is_causal=True)[0]
    return o.transpose(0, 1).to(torch.bfloat16)


def flat_loss(L, model, prompt_len, branch_len, prompt_tok, resp_tok):
    """Every (prompt, response) pair as its own sequence: the prompt is recomputed for each branch."""
    total, p0, r0 = 0.0, 0, 0
    for P, rs in zip(prompt_len, branch_len):
        for r in rs:
            tok = torch.cat([prompt_tok[p0:p0 + P], resp_tok[r0:r0 + r]])
            pos = torch.arange(P + r, device=tok.device)
            x = model.emb[tok]
            for layer in model.layers:
                q, k, v = layer.qkv(x, pos)
                x = layer.after_attention(x, causal_attention_reference(q, k, v))
            h = L.rms_norm(x, model.norm)[P - 1:P + r - 1]          # states that predict the response tokens
            logits = F.linear(h.to(torch.bfloat16), model.head.to(torch.bfloat16)).float()
            total = total + F.cross_entropy(logits, resp_tok[r0:r0 + r], reduction="sum")
            r0 += r
        p0 += P
    return total


@pytest.mark.parametrize("D", [64, 96])
def test_tree_and_flattened_training_agree(mods, D):
    B, L = mods
    torch.manual_seed(11)
    prompt_len, branch_len = [300, 129], [[130, 64, 257, 1], [200, 33]]
    plan = B.Plan(prompt_len, branch_len, H_Q, H_KV, D, device=0)
    g = torch.Generator().manual_seed(3)
    prompt_tok = torch.randint(0, VOCAB, (sum(prompt_len),), generator=g).cuda()
    resp_tok = torch.randint(0, VOCAB, (sum(sum(b) for b in branch_len),), generator=g).cuda()
    tree_model = TinyLM(L, D).cuda()
    flat_model = copy.deepcopy(tree_model)

    # ---- one step: loss and the gradient of every weight
    lt = tree_loss(L, tree_model, plan, prompt_tok, resp_tok)
    lf = flat_loss(L, flat_model, prompt_len, branch_len, prompt_tok, resp_tok)
    lt.backward()
    lf.backward()
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    n_tok = resp_tok.numel()
    assert abs(lt.item() - lf.item()) <= 2e-3 * abs(lf.item()), (lt.item() / n_tok, lf.item() / n_tok)
    worst = {}
    for (name, pt), (_, pf) in zip(tree_model.named_parameters(), flat_model.named_parameters()):
        rel = ((pt.grad - pf.grad).norm() / pf.grad.norm()).item()
        worst[name] = rel
        # both sides round P and dS to bf16 in their attention, at different places: a few 1e-3 per tensor
        assert rel <= 2e-2, (name, rel)
    print("largest relative gradient difference:", max(worst, key=worst.get), max(worst.values()))

    # ---- loss trajectory over a few plain SGD steps on both copies
    opt_t = torch.optim.SGD(tree_model.parameters(), lr=2e-3)
    opt_f = torch.optim.SGD(flat_model.parameters(), lr=2e-3)
    traj = []
    for step in range(4):
        if step:
            opt_t.zero_grad(); opt_f.zero_grad()
            lt = tree_loss(L, tree_model, plan, prompt_tok, resp_tok)
            lf = flat_loss(L, flat_model, prompt_len, branch_len, prompt_tok, resp_tok)
            lt.backward(); lf.backward()
        opt_t.step(); opt_f.step()
        traj.append((lt.item() / n_tok, lf.item() / n_tok))
    print("loss per token (tree, flattened):", traj)
    assert traj[-1][1] < traj[0][1]                                   # the steps do train
    for a, b in traj:
        assert abs(a - b) <= 2e-3 * abs(b), traj


def test_seam_index_and_positions(mods):
    B, L = mods
    plan = B.Plan([5, 3], [[2, 1], [3]], 4, 2, 64, device=0)
    pos_p, pos_r = L.tree_positions(plan)
    assert pos_p.tolist() == [0, 1, 2, 3, 4, 0, 1, 2] and pos_r.tolist() == [5, 6, 5, 3, 4, 5]
    from_prompt, index = L.seam_index(plan)
    assert from_prompt.tolist() == [True, False, True, True, False, False]
    assert index.tolist() == [4, 0, 4, 7, 3, 4]
