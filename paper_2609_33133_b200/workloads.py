"""Seeded synthetic workloads: lengths and tensors only, none of the method's arithmetic.

Both the CUDA path and the CPU oracle receive their inputs from here (the
tests hand the same arrays to each), so this module must stay free of any
attention maths.  It stands in for the paper's four post-training corpora
(Sec. 4.1), copying only their regimes: prompt-heavy, response-heavy, mixed,
G = 8 by default, Qwen2.5-7B attention geometry (28 query heads, 4 KV heads,
head dimension 128).

Lengths for the log-normal configurations come from a self-contained counter
generator (splitmix64 -> Box-Muller in float64), so they do not depend on any
library's random stream:  len = clip(rint(median * exp(sigma * z)), lo, hi).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List

import numpy as np
import torch

_MASK64 = (1 << 64) - 1


def _splitmix64(state: int):
    state = (state + 0x9E3779B97F4A7C15) & _MASK64
    z = state
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return state, z ^ (z >> 31)


class CounterNormal:
    """Standard normal deviates from splitmix64 + Box-Muller (cosine branch)."""

    def __init__(self, seed: int):
        self.state = seed & _MASK64

    def _uniform(self) -> float:
        self.state, z = _splitmix64(self.state)
        return ((z >> 11) + 0.5) / float(1 << 53)

    def normal(self) -> float:
        u1, u2 = self._uniform(), self._uniform()
        return math.sqrt(-2.0 * math.log(u1)) * math.cos(2.0 * math.pi * u2)

    def lognormal_len(self, median: float, sigma: float, lo: int, hi: int) -> int:
        x = median * math.exp(sigma * self.normal())
        return int(min(max(int(round(x)), lo), hi))


@dataclass
class Workload:
    name: str
    prompt_len: List[int]
    branch_len: List[List[int]]
    h_q: int
    h_kv: int
    head_dim: int
    seed: int
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def n_groups(self):
        return len(self.prompt_len)

    @property
    def total_prompt(self):
        return sum(self.prompt_len)

    @property
    def total_response(self):
        return sum(sum(b) for b in self.branch_len)

    def flattened(self) -> "Workload":
        """The no-reuse form: every branch becomes its own linear sequence [P; R_i]."""
        seqs = []
        for p, bl in zip(self.prompt_len, self.branch_len):
            for r in (bl if bl else [0]):
                seqs.append(p + r)
        return Workload(self.name + "-flattened", seqs, [[] for _ in seqs], self.h_q, self.h_kv,
                        self.head_dim, self.seed, "prompt duplicated per branch")


def config(index: int, scale_down: int = 1) -> Workload:
    """The five configurations of the benchmark contract, 1-based.

    scale_down divides every length (not the group or head counts); it is used
    by tests that need the shape of a configuration at a size the oracle
    finishes quickly.
    """
    s = scale_down
    if index == 1:
        return Workload("cfg1-small", [256 // s], [[128 // s] * 4], 4, 4, 64, 1001)
    if index == 2:
        return Workload("cfg2-7b-layer", [8192 // s], [[2048 // s] * 8], 28, 4, 128, 1002)
    if index == 3:
        return Workload("cfg3-prompt-dominated", [65536 // s] * 2, [[1024 // s] * 8] * 2, 32, 8, 128, 1003,
                        extra={"force_split": True})
    if index == 4:
        rng = CounterNormal(4)
        bl = [[rng.lognormal_len(8192 / s, 0.6, max(512 // s, 1), 32768 // s) for _ in range(16)] for _ in range(4)]
        return Workload("cfg4-response-dominated", [1024 // s] * 4, bl, 32, 8, 128, 1004)
    if index == 5:
        rng = CounterNormal(5)
        pl, bl = [], []
        for _ in range(32):
            pl.append(rng.lognormal_len(2048 / s, 1.2, max(256 // s, 1), 32768 // s))
            bl.append([rng.lognormal_len(2048 / s, 1.0, max(64 // s, 1), 16384 // s) for _ in range(8)])
        return Workload("cfg5-mixed-packed", pl, bl, 32, 8, 128, 1005)
    raise ValueError("config index must be 1..5")


def config5_prefix_256k() -> Workload:
    """Shortest prefix of configuration 5's groups whose tree tokens reach 262144."""
    w = config(5)
    tot, n = 0, 0
    while n < w.n_groups and tot < 262144:
        tot += w.prompt_len[n] + sum(w.branch_len[n])
        n += 1
    return Workload("cfg5b-256k-prefix", w.prompt_len[:n], w.branch_len[:n], w.h_q, w.h_kv, w.head_dim, 1005)


TENSOR_NAMES = ("q_p", "k_p", "v_p", "do_p", "q_r", "k_r", "v_r", "do_r")


# --------------------------------------------------------------------------- #
# Sharding over GPUs without any exchange step.  Replay trees are independent of
# each other (data-parallel replicas work on different trees, Sec. 3.5) and, inside
# attention, so are KV heads: a KV head with the query heads that read it can live
# on one GPU, and the many-to-one prompt-KV gradient of Eq. 2 stays local to it.
# So the units are whole groups when there are at least as many groups as ranks,
# and (group, KV head) pairs otherwise; they are dealt out largest first by visible
# (query, key) pairs, each to the rank with the least work so far.
@dataclass
class Part:
    """Some groups of a workload, restricted to some of its KV heads (and their query heads)."""
    groups: List[int]
    kv_heads: List[int]


def _group_pairs(w: Workload, g: int) -> int:
    tri = lambda n: n * (n + 1) // 2
    p = w.prompt_len[g]
    return tri(p) + sum(r * p + tri(r) for r in w.branch_len[g])


def partition(w: Workload, world: int) -> List[List[Part]]:
    """Parts per rank.  Every (group, KV head) of `w` lands in exactly one part of exactly one rank."""
    all_heads = list(range(w.h_kv))
    if w.n_groups >= world:
        units = [(g, None) for g in range(w.n_groups)]
        weight = lambda u: _group_pairs(w, u[0]) * w.h_kv
    else:
        units = [(g, c) for g in range(w.n_groups) for c in all_heads]
        weight = lambda u: _group_pairs(w, u[0])
    order = sorted(range(len(units)), key=lambda i: (-weight(units[i]), i))
    load = [0] * world
    mine: List[List[tuple]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        mine[r].append(units[i])
        load[r] += weight(units[i])
    shards = []
    for r in range(world):
        whole = sorted(g for g, c in mine[r] if c is None)
        parts = [Part(whole, all_heads)] if whole else []
        by_heads = {}
        for g in sorted({g for g, c in mine[r] if c is not None}):
            heads = tuple(sorted(c for gg, c in mine[r] if gg == g and c is not None))
            by_heads.setdefault(heads, []).append(g)
        parts += [Part(gs, list(heads)) for heads, gs in sorted(by_heads.items())]
        shards.append(parts)
    return shards


def part_workload(w: Workload, part: Part) -> Workload:
    rep = w.h_q // w.h_kv
    return Workload(f"{w.name}[g{part.groups},kv{part.kv_heads}]", [w.prompt_len[g] for g in part.groups],
                    [list(w.branch_len[g]) for g in part.groups], rep * len(part.kv_heads), len(part.kv_heads), w.head_dim,
                    w.seed, w.note, dict(w.extra))


def _part_index(w: Workload, part: Part):
    """(prompt token index, response token index, query head index, KV head index) of a part inside `w`."""
    cu_p = np.concatenate([[0], np.cumsum(w.prompt_len)])
    flat = [sum(b) for b in w.branch_len]
    cu_r = np.concatenate([[0], np.cumsum(flat)])
    tok_p = np.concatenate([np.arange(cu_p[g], cu_p[g + 1]) for g in part.groups]) if part.groups else np.zeros(0, int)
    tok_r = np.concatenate([np.arange(cu_r[g], cu_r[g + 1]) for g in part.groups]) if part.groups else np.zeros(0, int)
    rep = w.h_q // w.h_kv
    hq = np.concatenate([np.arange(c * rep, (c + 1) * rep) for c in part.kv_heads])
    return tok_p.astype(np.int64), tok_r.astype(np.int64), hq.astype(np.int64), np.asarray(part.kv_heads, dtype=np.int64)


def part_tensors(w: Workload, t, part: Part):
    """The part's slices of a workload's tensors (copies; pure data movement)."""
    tok_p, tok_r, hq, hkv = _part_index(w, part)
    out = {}
    for name in TENSOR_NAMES:
        x = t[name]
        tok = torch.as_tensor(tok_p if name.endswith("_p") else tok_r, device=x.device)
        heads = torch.as_tensor(hq if name[0] in "qd" else hkv, device=x.device)
        out[name] = x.index_select(0, tok).index_select(1, heads).contiguous()
    return out


def scatter_part(w: Workload, part: Part, part_out, full_out):
    """Writes a part's outputs (any of o_*, lse_*, dq_*, dk_*, dv_*) into full-size tensors of `w`."""
    tok_p, tok_r, hq, hkv = _part_index(w, part)
    for name, x in part_out.items():
        if name not in full_out:
            continue
        dst = full_out[name]
        tok = torch.as_tensor(tok_p if name.endswith("_p") else tok_r, device=dst.device)
        q_like = name.startswith(("o_", "lse_", "dq_"))
        heads = torch.as_tensor(hq if q_like else hkv, device=dst.device)
        if name.startswith("lse"):
            dst[heads[:, None], tok[None, :]] = x.to(dst.device)
        else:
            dst[tok[:, None], heads[None, :]] = x.to(dst.device)


def make_tensors(w: Workload, device="cpu"):
    """bf16 tensors ~ N(0,1) for a workload, from torch's seeded generator.

    Generated on `device` ('cpu' for anything the oracle will look at in full;
    'cuda' for the large benchmark shapes, whose bits can still be copied back
    for spot checks).  Order of generation is fixed: TENSOR_NAMES.
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed)
    tp, tr = w.total_prompt, w.total_response
    shapes = {
        "q_p": (tp, w.h_q), "k_p": (tp, w.h_kv), "v_p": (tp, w.h_kv), "do_p": (tp, w.h_q),
        "q_r": (tr, w.h_q), "k_r": (tr, w.h_kv), "v_r": (tr, w.h_kv), "do_r": (tr, w.h_q),
    }
    out = {}
    for name in TENSOR_NAMES:
        t, h = shapes[name]
        x = torch.randn((t, h, w.head_dim), generator=gen, device=device, dtype=torch.float32)
        out[name] = x.to(torch.bfloat16)
    return out


def flatten_tensors(w: Workload, t):
    """Inputs of the flattened baseline: [P; R_i] per branch, prompt rows duplicated.

    The prompt rows' dO is divided by the branch count so that the copies'
    prompt seeds add up to the tree's dO_P.  Pure data movement plus that one
    scaling; returned as the 'prompt' tensors of `w.flattened()`.
    """
    qs, ks, vs, dos = [], [], [], []
    cu_p = np.concatenate([[0], np.cumsum(w.prompt_len)])
    r_off = 0
    for g, bl in enumerate(w.branch_len):
        p0, p1 = int(cu_p[g]), int(cu_p[g + 1])
        copies = max(len(bl), 1)
        for r in (bl if bl else [0]):
            qs += [t["q_p"][p0:p1], t["q_r"][r_off:r_off + r]]
            ks += [t["k_p"][p0:p1], t["k_r"][r_off:r_off + r]]
            vs += [t["v_p"][p0:p1], t["v_r"][r_off:r_off + r]]
            dos += [(t["do_p"][p0:p1].float() / copies).to(torch.bfloat16), t["do_r"][r_off:r_off + r]]
            r_off += r
    return {"q_p": torch.cat(qs), "k_p": torch.cat(ks), "v_p": torch.cat(vs), "do_p": torch.cat(dos)}
