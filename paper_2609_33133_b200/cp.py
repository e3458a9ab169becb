"""The two replay primitives of Sec. 3.3, MoveQ and TreeMoveKV, on top of the library's partial-state entry points.

MoveQ first; TreeMoveKV (lane-local KV rings under a replay-grid placement) at the end of the file.

Rank r of n keeps shard r of every group's prompt KV (stationary) and owns some response branches (their K/V,
their queries, their outputs).  Forward: the response queries of all branches are made known to every rank, each
rank computes every query's partial softmax state over its prompt-KV shard (plus, for the branches it owns, the
branch's own causal prefix), and the n states of a query are merged on its owner.  Backward: the merged output,
its LSE and the seed dO are made known to every rank; each rank computes its shard's dK_P / dV_P (complete: the
many-to-one sum of Eq. 2 is local to the shard's owner), dK_R / dV_R of the branches it owns, and its contribution
to every dQ; the dQ contributions are summed on the way back to the queries' owners (the forward exchange run in reverse).

The per-rank compute steps are calls into the library (`CudaBackend`: augtree_replay_fwd_state, augtree_merge_states,
augtree_replay_bwd_state); what remains here is bookkeeping and the exchange steps.  `moveq_emulate` runs all ranks
in one process on one GPU, phase by phase; `moveq_rank` is one rank of a multi-process run over torch.distributed
(NCCL on GPUs; the CPU tests drive it over gloo with a stand-in compute backend).  The exchange is written with
whole-tensor collectives (all_reduce of row-disjoint tensors, all_gather of states) for clarity; a deployment would
send each owner only its rows (all-to-all of states, reduce-scatter of dQ) as NVLink peer copies.  No collective or
copy here uses multicast loads.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List

import numpy as np
import torch


def shard_bounds(length: int, n: int):
    """n contiguous token ranges covering [0, length), sizes differing by at most one (length >= n)."""
    if length < n:
        raise ValueError("a prompt needs at least one token per rank")
    cuts = [(length * i) // n for i in range(n + 1)]
    return [(cuts[i], cuts[i + 1]) for i in range(n)]


@dataclass
class RankLayout:
    """Bookkeeping of one rank: which prompt tokens it holds and which branches it owns."""
    rank: int
    world: int
    prompt_idx: np.ndarray          # packed prompt-token indices of this rank's shards, group order
    shard_len: List[int]            # per group
    owned: List[int]                # global branch indices owned (branch i belongs to rank i % world)
    branch_tok: List[np.ndarray]    # per global branch: its packed response-token indices
    branch_group: List[int]


def make_layout(w, rank: int, world: int) -> RankLayout:
    cu_p = np.concatenate([[0], np.cumsum(w.prompt_len)]).astype(np.int64)
    idx, lens = [], []
    for g, P in enumerate(w.prompt_len):
        a, b = shard_bounds(P, world)[rank]
        idx.append(np.arange(cu_p[g] + a, cu_p[g] + b))
        lens.append(b - a)
    branch_tok, branch_group, off = [], [], 0
    for g, bl in enumerate(w.branch_len):
        for r in bl:
            branch_tok.append(np.arange(off, off + r))
            branch_group.append(g)
            off += r
    owned = [i for i in range(len(branch_tok)) if i % world == rank]
    return RankLayout(rank, world, np.concatenate(idx), lens, owned, branch_tok, branch_group)


def _branch_sets(lay: RankLayout):
    """(branches, include_own) for the two compute calls of a rank: the branches it owns, then the others."""
    others = [i for i in range(len(lay.branch_tok)) if i not in lay.owned]
    return [(s, own) for s, own in ((lay.owned, True), (others, False)) if s]


def _rows(lay: RankLayout, branches):
    return np.concatenate([lay.branch_tok[i] for i in branches])


def _branch_len_by_group(w, lay: RankLayout, branches):
    out = [[] for _ in w.prompt_len]
    for i in branches:
        out[lay.branch_group[i]].append(len(lay.branch_tok[i]))
    return out


class CudaBackend:
    """The per-rank compute steps as library calls.  A call is described by the lengths of the key shards it holds (one
    per group) and of the response branches it is given (per group); plans are cached by that description."""

    def __init__(self, binding, w, device=0):
        self.B, self.w, self.device, self._plans = binding, w, device, {}

    def _plan(self, shard_len, branch_lens):
        key = (tuple(shard_len), tuple(tuple(b) for b in branch_lens))
        if key not in self._plans:
            w = self.w
            self._plans[key] = self.B.Plan(list(shard_len), [list(b) for b in branch_lens], w.h_q, w.h_kv, w.head_dim, device=self.device)
        return self._plans[key]

    def _ws(self, plan):
        return torch.empty(max(plan.ws_fwd_bytes, plan.ws_bwd_bytes, 256), device="cuda", dtype=torch.uint8)

    def fwd_state_on(self, shard_len, branch_lens, include_own, q, k_r, v_r, k_p, v_p):
        plan = self._plan(shard_len, branch_lens)
        so = torch.empty((plan.total_r, self.w.h_q, self.w.head_dim), device="cuda", dtype=torch.float32)
        sl = torch.empty((self.w.h_q, plan.total_r), device="cuda", dtype=torch.float32)
        plan.replay_fwd_state(q, k_r, v_r, k_p, v_p, so, sl, include_own, self._ws(plan))
        return so, sl

    def merge(self, _unused, states_o, states_lse):
        n = states_o[0].shape[0]
        plan = self._plan([1], [[n]])                     # the merge only needs the row count and the head geometry
        o = torch.empty((n, self.w.h_q, self.w.head_dim), device="cuda", dtype=torch.bfloat16)
        lse = torch.empty((self.w.h_q, n), device="cuda", dtype=torch.float32)
        plan.merge_states(states_o, states_lse, o, lse)
        return o, lse

    def bwd_state_on(self, shard_len, branch_lens, include_own, q, k_r, v_r, k_p, v_p, o, lse, do, dkp, dvp):
        plan = self._plan(shard_len, branch_lens)
        hq, hkv, d = self.w.h_q, self.w.h_kv, self.w.head_dim
        dq = torch.empty((plan.total_r, hq, d), device="cuda", dtype=torch.float32)
        dk = torch.empty((plan.total_r, hkv, d), device="cuda", dtype=torch.bfloat16)
        dv = torch.empty_like(dk)
        plan.replay_bwd_state(q, k_r, v_r, k_p, v_p, o, lse, do, dq, dk, dv, dkp, dvp, include_own, self._ws(plan))
        return dq, dk, dv

    def fwd_state(self, lay, branches, include_own, *tensors):
        return self.fwd_state_on(lay.shard_len, _branch_len_by_group(self.w, lay, branches), include_own, *tensors)

    def bwd_state(self, lay, branches, include_own, *tensors):
        return self.bwd_state_on(lay.shard_len, _branch_len_by_group(self.w, lay, branches), include_own, *tensors)

    def status_ok(self):
        return all(p.device_status() == (0, 0) for p in self._plans.values())


def fwd_compute(backend, w, lay, q_all, k_r_all, v_r_all, k_p_shard, v_p_shard):
    """This rank's partial state of EVERY response query: (state_o [sumR,H_q,d], state_lse [H_q,sumR])."""
    tr = q_all.shape[0]
    so = torch.zeros((tr, w.h_q, w.head_dim), device=q_all.device, dtype=torch.float32)
    sl = torch.full((w.h_q, tr), float("-inf"), device=q_all.device, dtype=torch.float32)
    for branches, own in _branch_sets(lay):
        rows = torch.as_tensor(_rows(lay, branches), device=q_all.device)
        # K/V of the branches' own sequences are needed only where the rank owns them; elsewhere any buffer of the shape will do
        k_r = k_r_all.index_select(0, rows).contiguous()
        v_r = v_r_all.index_select(0, rows).contiguous()
        o_part, l_part = backend.fwd_state(lay, branches, own, q_all.index_select(0, rows).contiguous(), k_r, v_r, k_p_shard, v_p_shard)
        so[rows] = o_part
        sl[:, rows] = l_part
    return so, sl


def bwd_compute(backend, w, lay, q_all, k_r_all, v_r_all, k_p_shard, v_p_shard, o_all, lse_all, do_all):
    """This rank's gradient work: (dq contribution for every query fp32, dk_r / dv_r of owned branches scattered into
    full-size zero tensors, dK_P / dV_P of its prompt shards fp32)."""
    tr, dev = q_all.shape[0], q_all.device
    dq = torch.zeros((tr, w.h_q, w.head_dim), device=dev, dtype=torch.float32)
    dk_r = torch.zeros((tr, w.h_kv, w.head_dim), device=dev, dtype=torch.bfloat16)
    dv_r = torch.zeros_like(dk_r)
    dkp = torch.zeros((int(sum(lay.shard_len)), w.h_kv, w.head_dim), device=dev, dtype=torch.float32)
    dvp = torch.zeros_like(dkp)
    for branches, own in _branch_sets(lay):
        rows = torch.as_tensor(_rows(lay, branches), device=dev)
        sel = lambda x: x.index_select(0, rows).contiguous()
        dq_p, dk_p, dv_p = backend.bwd_state(lay, branches, own, sel(q_all), sel(k_r_all), sel(v_r_all), k_p_shard, v_p_shard,
                                             sel(o_all), lse_all.index_select(1, rows).contiguous(), sel(do_all), dkp, dvp)
        dq[rows] = dq_p
        if own:
            dk_r[rows] = dk_p
            dv_r[rows] = dv_p
    return dq, dk_r, dv_r, dkp, dvp


def moveq_emulate(binding, w, t, world: int, device=0):
    """All ranks of a MoveQ replay in one process on one GPU, phase by phase (each phase for every rank, then the
    exchange that follows it).  `t`: the workload's full tensors on the device.  Returns o_r, lse_r, dq_r, dk_r, dv_r
    and the prompt-KV gradient seeds dk_p, dv_p (fp32, replay part only: the prefill backward adds its own)."""
    backend = CudaBackend(binding, w, device)
    lays = [make_layout(w, r, world) for r in range(world)]
    shard = [(t["k_p"][torch.as_tensor(l.prompt_idx, device="cuda")].contiguous(),
              t["v_p"][torch.as_tensor(l.prompt_idx, device="cuda")].contiguous()) for l in lays]
    # forward: queries known everywhere (the exchange: all-gather of the owners' query rows) -> states -> merge on the owners
    states = [fwd_compute(backend, w, lays[r], t["q_r"], t["k_r"], t["v_r"], *shard[r]) for r in range(world)]
    o, lse = backend.merge(None, [s[0] for s in states], [s[1] for s in states])
    # backward: merged O, LSE and dO known everywhere -> per-rank gradients -> dQ summed back to the owners
    parts = [bwd_compute(backend, w, lays[r], t["q_r"], t["k_r"], t["v_r"], *shard[r], o, lse, t["do_r"]) for r in range(world)]
    dq = torch.stack([p[0] for p in parts]).sum(dim=0)            # the reverse exchange: sum over KV owners, fixed rank order
    dk_r = torch.stack([p[1].float() for p in parts]).sum(dim=0)  # every row has exactly one owner: the others hold zeros
    dv_r = torch.stack([p[2].float() for p in parts]).sum(dim=0)
    dk_p = torch.zeros((w.total_prompt, w.h_kv, w.head_dim), device="cuda", dtype=torch.float32)
    dv_p = torch.zeros_like(dk_p)
    for r in range(world):
        idx = torch.as_tensor(lays[r].prompt_idx, device="cuda")
        dk_p[idx] = parts[r][3]
        dv_p[idx] = parts[r][4]
    torch.cuda.synchronize()
    if not backend.status_ok():
        raise RuntimeError("device status")
    return {"o_r": o, "lse_r": lse, "dq_r": dq, "dk_r": dk_r, "dv_r": dv_r, "dk_p": dk_p, "dv_p": dv_p}


def moveq_rank(dist, backend, w, rank: int, world: int, local: Dict[str, torch.Tensor]):
    """One rank of a multi-process MoveQ replay.  `local`: k_p, v_p = this rank's prompt-KV shards (stationary), and
    q_r, k_r, v_r, do_r as full-size tensors that hold the rows of the branches this rank owns and zeros elsewhere.
    Returns, for the rows this rank owns (zeros elsewhere): o_r, lse_r, dq_r, dk_r, dv_r; and dk_p, dv_p of its shards."""
    lay = make_layout(w, rank, world)

    def everywhere(x):               # rows are owned by exactly one rank: a sum makes every rank hold all of them
        y = x.float().clone()
        dist.all_reduce(y, op=dist.ReduceOp.SUM)
        return y.to(x.dtype)

    q_all = everywhere(local["q_r"])                       # MoveQ's query movement
    so, sl = fwd_compute(backend, w, lay, q_all, local["k_r"], local["v_r"], local["k_p"], local["v_p"])
    states_o = [torch.empty_like(so) for _ in range(world)]
    states_l = [torch.empty_like(sl) for _ in range(world)]
    dist.all_gather(states_o, so)                          # partial states to the queries' owners
    dist.all_gather(states_l, sl)
    o_all, lse_all = backend.merge(None, states_o, states_l)
    do_all = everywhere(local["do_r"])
    dq_part, dk_r, dv_r, dkp, dvp = bwd_compute(backend, w, lay, q_all, local["k_r"], local["v_r"], local["k_p"], local["v_p"],
                                                o_all, lse_all, do_all)
    dist.all_reduce(dq_part, op=dist.ReduceOp.SUM)         # the forward exchange in reverse
    mine = torch.zeros(q_all.shape[0], dtype=torch.bool, device=q_all.device)
    if lay.owned:
        mine[torch.as_tensor(_rows(lay, lay.owned), device=q_all.device)] = True
    keep = lambda x, rows_first=True: x * (mine[:, None, None] if rows_first else mine[None, :]).to(x.dtype)
    return {"o_r": keep(o_all), "lse_r": keep(lse_all, False), "dq_r": keep(dq_part), "dk_r": dk_r, "dv_r": dv_r, "dk_p": dkp, "dv_p": dvp}


# --------------------------------------------------------------------------------------------------------------
# TreeMoveKV (Sec. 3.3): response-local move-KV.  The d ranks form s lanes of d_lane = d / s ranks; a placement X
# (Eq. 6, augtree_assign_grid) gives every response path a (round, lane) cell; a lane keeps the whole prompt KV,
# sharded over its d_lane ranks, and within a round each of its ranks owns some of the cell's paths whole (queries,
# response K/V and outputs never leave their rank: response-path locality).  Only the prompt-KV shards travel: in
# ring stage t rank r holds shard (r - t) mod d_lane, computes the partial state of its own queries over it and
# merges it into their running state; in the backward pass the shards go round once more with their fp32 dK_P / dV_P
# accumulators, every rank adds its queries' share (Eq. 2 accumulated along the ring) and keeps its dQ to itself.
def treemovekv_emulate(binding, w, t, s: int, d_lane: int, rounds: int = 1, device=0):
    """All ranks of a TreeMoveKV replay (s lanes x d_lane ranks, `rounds` rounds) in one process on one GPU, stage by
    stage.  One group only (a replay tree).  Returns the same tensors as moveq_emulate plus the placement used."""
    if w.n_groups != 1 or d_lane > 16:
        raise ValueError("one replay tree at a time, lanes of at most 16 ranks")
    P, R = w.prompt_len[0], w.branch_len[0]
    tiles = lambda r: -(-r // 128) * -(-P // 128) + (-(-r // 128)) * (-(-r // 128) + 1) // 2   # unit weight: valid tile count
    x_round, x_lane, _, _ = binding.assign_grid([tiles(r) for r in R], R, n_rounds=rounds, n_lanes=s)
    bounds = shard_bounds(P, d_lane)
    cu_r = np.concatenate([[0], np.cumsum(R)]).astype(np.int64)
    hq, hkv, d = w.h_q, w.h_kv, w.head_dim
    dev = "cuda"
    kp = [t["k_p"][a:b].contiguous() for a, b in bounds]
    vp = [t["v_p"][a:b].contiguous() for a, b in bounds]
    out = {"o_r": torch.zeros((w.total_response, hq, d), device=dev, dtype=torch.bfloat16),
           "lse_r": torch.zeros((hq, w.total_response), device=dev, dtype=torch.float32),
           "dq_r": torch.zeros((w.total_response, hq, d), device=dev, dtype=torch.float32),
           "dk_r": torch.zeros((w.total_response, hkv, d), device=dev, dtype=torch.bfloat16),
           "dv_r": torch.zeros((w.total_response, hkv, d), device=dev, dtype=torch.bfloat16),
           "dk_p": torch.zeros((P, hkv, d), device=dev, dtype=torch.float32),
           "dv_p": torch.zeros((P, hkv, d), device=dev, dtype=torch.float32)}
    plans = []
    for rnd in range(rounds):
        for lane in range(s):
            cell = [k for k in range(len(R)) if x_round[k] == rnd and x_lane[k] == lane]
            # every lane holds its own copy of the prompt-KV shards, and so its own accumulators for them
            acc = [(torch.zeros((b - a, hkv, d), device=dev, dtype=torch.float32), torch.zeros((b - a, hkv, d), device=dev, dtype=torch.float32))
                   for a, b in bounds]
            for r in range(d_lane):
                mine = [k for i, k in enumerate(cell) if i % d_lane == r]
                if not mine:
                    continue
                rows = torch.as_tensor(np.concatenate([np.arange(cu_r[k], cu_r[k + 1]) for k in mine]), device=dev)
                sel = lambda x: x.index_select(0, rows).contiguous()
                q, k_r, v_r, do = sel(t["q_r"]), sel(t["k_r"]), sel(t["v_r"]), sel(t["do_r"])
                stage_plans = [binding.Plan([b - a], [[R[k] for k in mine]], hq, hkv, d, device=device) for a, b in bounds]
                plans += stage_plans
                ws = torch.empty(max(max(p.ws_fwd_bytes, p.ws_bwd_bytes) for p in stage_plans) + 256, device=dev, dtype=torch.uint8)
                n = int(rows.numel())
                # forward ring: one partial state per stage (stage 0: the rank's own shard and the paths' own causal
                # prefixes); the merge is associative, so the d_lane states are folded once, after the last stage
                states_o, states_l = [], []
                for stage in range(d_lane):
                    j = (r - stage) % d_lane
                    so = torch.empty((n, hq, d), device=dev, dtype=torch.float32)
                    sl = torch.empty((hq, n), device=dev, dtype=torch.float32)
                    stage_plans[j].replay_fwd_state(q, k_r, v_r, kp[j], vp[j], so, sl, stage == 0, ws)
                    states_o.append(so); states_l.append(sl)
                o = torch.empty((n, hq, d), device=dev, dtype=torch.bfloat16)
                lse = torch.empty((hq, n), device=dev, dtype=torch.float32)
                stage_plans[0].merge_states(states_o, states_l, o, lse)
                # backward ring: shards come round again with their accumulators
                dq = torch.zeros((n, hq, d), device=dev, dtype=torch.float32)
                dk = torch.empty((n, hkv, d), device=dev, dtype=torch.bfloat16)
                dv = torch.empty_like(dk)
                for stage in range(d_lane):
                    j = (r - stage) % d_lane
                    part = torch.empty((n, hq, d), device=dev, dtype=torch.float32)
                    stage_plans[j].replay_bwd_state(q, k_r, v_r, kp[j], vp[j], o, lse, do, part, dk, dv, acc[j][0], acc[j][1], stage == 0, ws)
                    dq += part
                out["o_r"][rows], out["dq_r"][rows], out["dk_r"][rows], out["dv_r"][rows] = o, dq, dk, dv
                out["lse_r"][:, rows] = lse
            # the lanes' copies of the prompt-KV gradient are summed when the prefill graphs are joined (Eq. 2 over lanes)
            for (a, b), (gk, gv) in zip(bounds, acc):
                out["dk_p"][a:b] += gk
                out["dv_p"][a:b] += gv
    torch.cuda.synchronize()
    if any(p.device_status() != (0, 0) for p in plans):
        raise RuntimeError("device status")
    out["placement"] = (x_round, x_lane)
    return out


def _ring_pass(dist, rank, world, tensors):
    """One ring step: every tensor of `tensors` goes to rank + 1 and is replaced by what rank - 1 sends.  Shapes may differ
    from rank to rank (shards differ by a token), so the sizes are exchanged with the data: first dimension only."""
    nxt, prv = (rank + 1) % world, (rank - 1) % world
    n_out = torch.tensor([t.shape[0] for t in tensors], dtype=torch.int64)
    n_in = torch.empty_like(n_out)
    for req in dist.batch_isend_irecv([dist.P2POp(dist.isend, n_out, nxt), dist.P2POp(dist.irecv, n_in, prv)]):
        req.wait()
    recv = [torch.empty((int(n),) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device) for n, t in zip(n_in.tolist(), tensors)]
    ops = [dist.P2POp(dist.isend, t.contiguous(), nxt) for t in tensors] + [dist.P2POp(dist.irecv, r, prv) for r in recv]
    for req in dist.batch_isend_irecv(ops):
        req.wait()
    return recv


def treemovekv_rank(dist, backend, w, rank: int, world: int, local: Dict[str, torch.Tensor]):
    """One rank of a multi-process TreeMoveKV lane (the whole process group is one lane, one round, one replay tree).
    `local`: k_p, v_p = this rank's prompt-KV shard; q_r, k_r, v_r, do_r = the rows of the branches it owns (branch k
    belongs to rank k % world), packed in branch order.  The prompt-KV shards go round the ring twice: once for the
    forward states, once more with their fp32 gradient accumulators, which are home again after the last step.
    Returns o_r, lse_r, dq_r, dk_r, dv_r for the owned rows and dk_p, dv_p of the rank's own shard."""
    if w.n_groups != 1:
        raise ValueError("one replay tree at a time")
    mine = [[r for k, r in enumerate(w.branch_len[0]) if k % world == rank]]
    q, k_r, v_r, do = local["q_r"], local["k_r"], local["v_r"], local["do_r"]
    have = bool(mine[0])
    kp, vp = local["k_p"], local["v_p"]
    states_o, states_l = [], []
    for stage in range(world):                              # forward ring
        if have:
            so, sl = backend.fwd_state_on([kp.shape[0]], mine, stage == 0, q, k_r, v_r, kp, vp)
            states_o.append(so); states_l.append(sl)
        kp, vp = _ring_pass(dist, rank, world, [kp, vp])   # after `world` passes the own shard is back
    res = {}
    if have:
        o, lse = backend.merge(None, states_o, states_l)
        dq = torch.zeros(q.shape, dtype=torch.float32, device=q.device)
    gk = torch.zeros(kp.shape, dtype=torch.float32, device=kp.device)
    gv = torch.zeros_like(gk)
    for stage in range(world):                              # backward ring: shards travel with their accumulators
        if have:
            part, dk, dv = backend.bwd_state_on([kp.shape[0]], mine, stage == 0, q, k_r, v_r, kp, vp, o, lse, do, gk, gv)
            dq += part
            if stage == 0:
                res.update(dk_r=dk, dv_r=dv)
        kp, vp, gk, gv = _ring_pass(dist, rank, world, [kp, vp, gk, gv])
    if have:
        res.update(o_r=o, lse_r=lse, dq_r=dq)
    res.update(dk_p=gk, dv_p=gv)
    return res
