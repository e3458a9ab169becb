"""MoveQ's exchange steps (Sec. 3.3) on two gloo ranks, with a stand-in compute backend.

The library's kernels need a GPU; what runs here is everything around them: who holds which prompt-KV shard, which
branches a rank owns, which calls include a branch's own causal prefix, the gathering of states to the merge, and the
reverse sum of the dQ contributions.  The compute steps are taken by a backend written from the oracle's
partial-state functions (fp64), so the assembled result must equal the oracle's full tree attention.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import tree_attention as ora
from paper_2609_33133_b200 import cp, workloads as wl

W = wl.Workload("moveq-gloo", [37, 12], [[9, 20, 5], [16]], 4, 2, 16, 5)


class OracleBackend:
    """fwd_state / merge / bwd_state of cp.CudaBackend, from the oracle's partial-state functions, on CPU."""

    def __init__(self, w):
        self.w, self.scale, self.rep = w, 1.0 / np.sqrt(w.head_dim), w.h_q // w.h_kv

    @staticmethod
    def _walk(shard_len, branch_lens):
        """(rows of the call's packed query tensor, rows of the call's key-shard tensor) branch by branch, group-major."""
        off_p = np.concatenate([[0], np.cumsum(shard_len)])
        pos = 0
        for g, lens in enumerate(branch_lens):
            for n in lens:
                yield slice(pos, pos + n), slice(int(off_p[g]), int(off_p[g + 1]))
                pos += n

    def fwd_state(self, lay, branches, include_own, *tensors):
        return self.fwd_state_on(lay.shard_len, cp._branch_len_by_group(self.w, lay, branches), include_own, *tensors)

    def bwd_state(self, lay, branches, include_own, *tensors):
        return self.bwd_state_on(lay.shard_len, cp._branch_len_by_group(self.w, lay, branches), include_own, *tensors)

    def fwd_state_on(self, shard_len, branch_lens, include_own, q, k_r, v_r, k_p, v_p):
        f = lambda x: x.double().numpy()
        q, k_r, v_r, k_p, v_p = f(q), f(k_r), f(v_r), f(k_p), f(v_p)
        so = np.zeros((q.shape[0], self.w.h_q, self.w.head_dim)); sl = np.zeros((self.w.h_q, q.shape[0]))
        for rows, shard in self._walk(shard_len, branch_lens):
            n = rows.stop - rows.start
            for h in range(self.w.h_q):
                c = h // self.rep
                st = ora.partial_state(q[rows, h], k_p[shard, c], v_p[shard, c], np.ones((n, shard.stop - shard.start), bool), self.scale)
                if include_own:
                    own = ora.partial_state(q[rows, h], k_r[rows, c], v_r[rows, c], np.tril(np.ones((n, n), bool)), self.scale)
                    st = ora.merge_states(st, own)
                o, lse = ora.finalize_state(st)
                so[rows, h], sl[h, rows] = o, lse
        return torch.from_numpy(so).float(), torch.from_numpy(sl).float()

    def merge(self, _plan, states_o, states_lse):
        acc = None
        for o, l in zip(states_o, states_lse):
            # a finalised state (o, lse) is the state (m = lse, l = 1, O_acc = o), head by head
            st = [(l[h].double().numpy(), np.ones(l.shape[1]), o[:, h].double().numpy()) for h in range(self.w.h_q)]
            acc = st if acc is None else [ora.merge_states(a, b) for a, b in zip(acc, st)]
        fin = [ora.finalize_state(s) for s in acc]
        o = np.stack([x[0] for x in fin], axis=1); lse = np.stack([x[1] for x in fin], axis=0)
        return torch.from_numpy(o).to(torch.bfloat16), torch.from_numpy(lse).float()

    def bwd_state_on(self, shard_len, branch_lens, include_own, q, k_r, v_r, k_p, v_p, o, lse, do, dkp, dvp):
        f = lambda x: x.double().numpy()
        q, k_r, v_r, k_p, v_p, o, lse, do = f(q), f(k_r), f(v_r), f(k_p), f(v_p), f(o), f(lse), f(do)
        dq = np.zeros_like(q); dk = np.zeros_like(k_r); dv = np.zeros_like(v_r)
        gk = np.zeros_like(k_p); gv = np.zeros_like(v_p)
        for rows, shard in self._walk(shard_len, branch_lens):
            n = rows.stop - rows.start
            for h in range(self.w.h_q):
                c = h // self.rep
                delta = (do[rows, h] * o[rows, h]).sum(axis=1, keepdims=True)
                parts = [(k_p[shard, c], v_p[shard, c], np.ones((n, shard.stop - shard.start), bool), "p")]
                if include_own:
                    parts.append((k_r[rows, c], v_r[rows, c], np.tril(np.ones((n, n), bool)), "r"))
                for k, v, vis, kind in parts:
                    p = np.where(vis, np.exp(self.scale * (q[rows, h] @ k.T) - lse[h, rows][:, None]), 0.0)
                    ds = p * (do[rows, h] @ v.T - delta)
                    dq[rows, h] += self.scale * (ds @ k)
                    if kind == "p":
                        gk[shard, c] += self.scale * (ds.T @ q[rows, h]); gv[shard, c] += p.T @ do[rows, h]
                    else:
                        dk[rows, c] += self.scale * (ds.T @ q[rows, h]); dv[rows, c] += p.T @ do[rows, h]
        dkp += torch.from_numpy(gk).float(); dvp += torch.from_numpy(gv).float()
        return torch.from_numpy(dq).float(), torch.from_numpy(dk).to(torch.bfloat16), torch.from_numpy(dv).to(torch.bfloat16)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t = wl.make_tensors(W)
    lay = cp.make_layout(W, rank, world)
    mine = torch.zeros(W.total_response, dtype=torch.bool)
    for i in lay.owned:
        mine[torch.as_tensor(lay.branch_tok[i])] = True
    idx = torch.as_tensor(lay.prompt_idx)
    local = {k: t[k] * mine[:, None, None].to(t[k].dtype) for k in ("q_r", "k_r", "v_r", "do_r")}   # a rank holds its own branches only
    local.update(k_p=t["k_p"][idx].contiguous(), v_p=t["v_p"][idx].contiguous())
    res = cp.moveq_rank(dist, OracleBackend(W), W, rank, world, local)
    out.put((rank, {k: v.float().numpy() for k, v in res.items()}, lay.prompt_idx))
    dist.barrier()
    dist.destroy_process_group()


def test_moveq_exchange_on_two_gloo_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    t = wl.make_tensors(W)
    tb = ora.TreeBatch(W.prompt_len, W.branch_len, W.h_q, W.h_kv, W.head_dim)
    f = lambda x: x.float().numpy().astype(np.float64)
    zero = np.zeros_like(f(t["do_p"]))
    ref = ora.tree_attention_fwd_bwd(tb, f(t["q_p"]), f(t["k_p"]), f(t["v_p"]), zero, f(t["q_r"]), f(t["k_r"]), f(t["v_r"]), f(t["do_r"]))
    # rows are owned by exactly one rank and zero elsewhere: the sum over ranks is the whole tensor
    for k, tol in (("o_r", 2e-2), ("lse_r", 1e-5), ("dq_r", 1e-2), ("dk_r", 5e-2), ("dv_r", 5e-2)):
        got = sum(r[1][k] for r in res)
        assert np.abs(got - ref[k]).max() <= tol, (k, np.abs(got - ref[k]).max())
    # each rank's prompt-KV gradients are those of its own shards (Eq. 2 is local to the shard's owner); with dO_P = 0
    # the oracle's dk_p / dv_p are exactly the replay seeds
    for rank, out, idx in res:
        assert np.abs(out["dk_p"] - ref["dk_p"][idx]).max() <= 1e-2 and np.abs(out["dv_p"] - ref["dv_p"][idx]).max() <= 1e-2
    covered = np.sort(np.concatenate([r[2] for r in res]))
    assert np.array_equal(covered, np.arange(W.total_prompt))


W_RING = wl.Workload("tmkv-gloo", [41], [[9, 20, 5, 16, 7]], 4, 2, 16, 6)


def _ring_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W_RING
    t = wl.make_tensors(w)
    cu = np.concatenate([[0], np.cumsum(w.branch_len[0])])
    rows = [np.arange(cu[k], cu[k + 1]) for k in range(len(w.branch_len[0])) if k % world == rank]
    rows = torch.as_tensor(np.concatenate(rows)) if rows else torch.zeros(0, dtype=torch.int64)
    a, b = cp.shard_bounds(w.prompt_len[0], world)[rank]
    local = {k: t[k][rows].contiguous() for k in ("q_r", "k_r", "v_r", "do_r")}
    local.update(k_p=t["k_p"][a:b].contiguous(), v_p=t["v_p"][a:b].contiguous())
    res = cp.treemovekv_rank(dist, OracleBackend(w), w, rank, world, local)
    out.put((rank, {k: v.float().numpy() for k, v in res.items()}, rows.numpy(), (a, b)))
    dist.barrier()
    dist.destroy_process_group()


def test_treemovekv_ring_on_three_gloo_ranks():
    """The lane-local KV ring of TreeMoveKV: prompt-KV shards passed from rank to rank (P2P send / receive), the states of
    a rank's own queries merged after the last stage, the shards' gradient accumulators home after a second round."""
    world, port = 3, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_ring_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = W_RING
    t = wl.make_tensors(w)
    tb = ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim)
    f = lambda x: x.float().numpy().astype(np.float64)
    ref = ora.tree_attention_fwd_bwd(tb, f(t["q_p"]), f(t["k_p"]), f(t["v_p"]), np.zeros_like(f(t["do_p"])), f(t["q_r"]), f(t["k_r"]),
                                     f(t["v_r"]), f(t["do_r"]))
    seen = []
    for rank, out, rows, (a, b) in res:
        seen += rows.tolist()
        for k, tol in (("o_r", 2e-2), ("dq_r", 1e-2), ("dk_r", 5e-2), ("dv_r", 5e-2)):
            assert np.abs(out[k] - ref[k][rows]).max() <= tol, (rank, k)
        assert np.abs(out["lse_r"] - ref["lse_r"][:, rows]).max() <= 1e-5
        # the accumulators that came home are those of the rank's own shard, summed over every rank's queries (Eq. 2)
        assert np.abs(out["dk_p"] - ref["dk_p"][a:b]).max() <= 1e-2 and np.abs(out["dv_p"] - ref["dv_p"][a:b]).max() <= 1e-2
    assert sorted(seen) == list(range(w.total_response))
