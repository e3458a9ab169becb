#!/usr/bin/env python
"""Benchmark of the tree-attention hot path (prefill + replay, forward + backward) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config I]

One "step" is one pass of the whole path over one batch of synthetic groups:
augtree_prefill_fwd -> augtree_replay_fwd -> augtree_replay_bwd -> augtree_prefill_bwd.
At N = 1 the workload is the 7B-shaped layer (configuration 2).  With N > 1 every
rank runs its own group of the same shape (independent trees shard with no
exchange step), so the scaling is weak and there is no data-path collective.

Prints one JSON line (rank 0).  `value` is useful TFLOP/s: causal-masked pairs
only, the prompt counted once, 14 * d FLOP per (query, key) pair and query head.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
from paper_2609_33133_b200 import workloads as wl  # noqa: E402

METRIC = "tree-attn fwd+bwd useful TFLOP/s (speedup vs flattened in 'flattened')"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_BF16_TFLOPS = 1590.0


def tri(n):
    return n * (n + 1) // 2


def pair_counts(w):
    pre = sum(tri(p) for p in w.prompt_len)
    rep = sum(r * p + tri(r) for p, bl in zip(w.prompt_len, w.branch_len) for r in bl)
    flat = sum(tri(p + r) for p, bl in zip(w.prompt_len, w.branch_len) for r in (bl if bl else [0]))
    return pre, rep, flat


def useful_flops(w):
    pre, rep, flat = pair_counts(w)
    per_pair = 14 * w.head_dim * w.h_q
    dh = w.head_dim * w.h_q
    # per kernel: the FLOPs its GEMMs execute (the two backward kernels both recompute S and dP:
    # 4 + 3 GEMMs for the 5 of the textbook backward; `total` counts the 5)
    return {"total": per_pair * (pre + rep), "prefill_fwd": 4 * dh * pre, "replay_fwd": 4 * dh * rep,
            "replay_bwd_dkdv": 8 * dh * rep, "prefill_bwd_dkdv": 8 * dh * pre, "replay_bwd_dq": 6 * dh * rep,
            "prefill_bwd_dq": 6 * dh * pre, "flattened_total": per_pair * flat, "reuse_factor": flat / (pre + rep)}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def ncu_dram_bytes(workload, kernel):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the latest ncu capture of this workload
    (profiles/ncu_dram_bytes.json, written from the capture whose command it records); None if not captured."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_bytes.json")
    try:
        return json.load(open(path)).get(workload, {}).get(kernel)
    except (OSError, ValueError):
        return None


def algorithmic_bytes(w, kernel):
    """HBM bytes a launch has to move if every tensor it touches crosses once (bf16 unless noted)."""
    d, hq, hkv = w.head_dim, w.h_q, w.h_kv
    tp, tr = w.total_prompt, w.total_response
    q = lambda n: 2 * n * hq * d            # a query-sized bf16 tensor
    kv = lambda n: 2 * n * hkv * d          # a key/value-sized bf16 tensor
    stats = lambda n: 8 * n * hq            # fp32 lse*log2e and delta per (row, head)
    return {
        "prefill_fwd": q(tp) + 2 * kv(tp) + q(tp) + 4 * tp * hq,
        "replay_fwd": q(tr) + 2 * kv(tr) + 2 * kv(tp) + q(tr) + 4 * tr * hq,
        # Q, dO, statistics, K/V of both tensors in; dK_R, dV_R out; fp32 prompt accumulators read and written
        "replay_bwd_dkdv": 2 * q(tr) + stats(tr) + 2 * kv(tr) + 2 * kv(tp) + 2 * kv(tr) + 2 * 2 * (2 * kv(tp)),
        "prefill_bwd_dkdv": 2 * q(tp) + stats(tp) + 2 * kv(tp) + 2 * 2 * (2 * kv(tp)),
        "replay_bwd_dq": 2 * q(tr) + stats(tr) + 2 * kv(tr) + 2 * kv(tp) + q(tr),
        "prefill_bwd_dq": 2 * q(tp) + stats(tp) + 2 * kv(tp) + q(tp),
    }[kernel]


def config_record(w, world):
    """The `config` object of the JSON line (the same keys for both arms)."""
    fl = useful_flops(w)
    return {"workload": w.name, "groups": w.n_groups, "prompt_tokens": w.total_prompt, "response_tokens": w.total_response,
            "h_q": w.h_q, "h_kv": w.h_kv, "head_dim": w.head_dim, "useful_tflop_per_step": fl["total"] / 1e12,
            "l2": "no flush: inputs + outputs exceed the 126 MB L2 (K/V reuse from L2 is part of the method)",
            "parallelism": f"independent groups x{world}"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- #
def oracle_sample(w, seconds_budget=20.0):
    """Times the fp64 oracle, as it stands, on whole (branch, query head) flattened
    sequences of the workload until the budget is used, and extrapolates to all of them."""
    from oracle import tree_attention as ora
    g = 0
    P, bl = w.prompt_len[g], w.branch_len[g]
    # tensors of group 0, one KV head and its first query head are enough for the sample
    gen = torch.Generator().manual_seed(w.seed)
    n_seq_total = sum(len(b) if b else 1 for b in w.branch_len) * w.h_q
    done, t_used, flops_flat = 0, 0.0, 0
    cores = len(os.sched_getaffinity(0))
    for r in (bl if bl else [0]):
        n = P + r
        q, k, v, do = (torch.randn((n, w.head_dim), generator=gen).to(torch.bfloat16).double().numpy() for _ in range(4))
        t0 = time.perf_counter()
        o, lse, p = ora.causal_attention_fwd(q, k, v, 1.0 / np.sqrt(w.head_dim))
        ora.causal_attention_bwd(q, k, v, o, p, do, 1.0 / np.sqrt(w.head_dim))
        t_used += time.perf_counter() - t0
        done += 1
        flops_flat += 14 * w.head_dim * tri(n)
        if t_used > seconds_budget:
            break
    # the sampled sequences stand for all (branch, head) sequences of the same group shape
    est_total_s = t_used / done * n_seq_total
    return {"seconds_sample": t_used, "sequences": done, "of": n_seq_total, "est_total_s": est_total_s, "cores": cores}


def run_reference(args, w):
    """--impl reference: the fp64 CPU oracle on a bounded sample per step."""
    fl = useful_flops(w)
    times = []
    info = None
    for i in range(args.warmup + args.steps):
        info = oracle_sample(w, seconds_budget=8.0)
        if i >= args.warmup:
            times.append(info["est_total_s"])
    est = statistics.mean(times)
    val = fl["total"] / est / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": est * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": config_record(w, 1),
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": info["cores"], "kind": "oracle",
                             "sample": f"{info['sequences']} of {info['of']} flattened (branch, head) sequences per step, time extrapolated"},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- #
def rank_workload(w, rank):
    """Rank r replays its own trees of the same shape: same lengths, seed + r (weak scaling, no exchange)."""
    return wl.Workload(w.name, w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, w.seed + rank, w.note, dict(w.extra))


def max_over_ranks(ms, dist, device="cuda"):
    """The job's time is the slowest rank's."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(flops_per_rank, world, ms_per_step):
    """Whole-job useful TFLOP/s: every rank does flops_per_rank in ms_per_step (the max over ranks)."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def time_steps(step_fn, steps, warmup, dist, sampler_index=None):
    """W warm-up steps, then K steps between two events, bracketed by barrier + synchronize; max over ranks."""
    for _ in range(warmup):
        step_fn()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    if sampler:
        sampler.__enter__()
        time.sleep(0.15)
    ev[0].record()
    for i in range(steps):
        step_fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    if sampler:
        sampler.__exit__()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    ms = max_over_ranks(ev[0].elapsed_time(ev[steps]), dist)
    time_steps.per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]  # this rank's, for median / min
    return ms, (sampler.summary() if sampler else None)


def measure_config(B, index, local_rank, steps=3, warmup=3, flattened=True):
    """One of the other configurations, briefly: tree step, flattened step, clocks (rank 0, N = 1 only)."""
    w = wl.config(index)
    fl = useful_flops(w)
    big = (w.total_prompt + w.total_response) * w.h_q * w.head_dim > 2e8
    t = {k: v.cuda() for k, v in wl.make_tensors(w, device="cuda" if big else "cpu").items()}
    splits = 4 if w.extra.get("force_split") else 0
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=local_rank, flags=B.FLAG_ZERO_PROMPT_GRAD,
                  kv_splits=splits)
    out = B.alloc_outputs(plan)
    ms, clocks = time_steps(lambda: B.run_forward_backward(plan, t, out), steps, warmup, None, sampler_index=local_rank)
    ms /= steps
    st = plan.device_status()
    if st != (0, 0):
        raise RuntimeError(f"device status {st} on configuration {index}")
    rec = {"workload": w.name, "tokens": w.total_prompt + w.total_response, "useful_tflop_per_step": fl["total"] / 1e12,
           "ms_per_step": ms, "tflops": fl["total"] / (ms * 1e-3) / 1e12, "steps": steps, "warmup": warmup,
           "reuse_factor": fl["reuse_factor"], "sm_mhz": clocks["sm_mhz"], "reasons": clocks["reasons"], "kv_splits": splits}
    del out
    if flattened:
        fw = w.flattened()
        ft = wl.flatten_tensors(w, t)
        del t
        e = lambda h: torch.empty((0, h, w.head_dim), dtype=torch.bfloat16, device="cuda")
        ft.update({"q_r": e(w.h_q), "k_r": e(w.h_kv), "v_r": e(w.h_kv), "do_r": e(w.h_q)})
        fplan = B.Plan(fw.prompt_len, fw.branch_len, fw.h_q, fw.h_kv, fw.head_dim, device=local_rank, flags=B.FLAG_ZERO_PROMPT_GRAD)
        fout = B.alloc_outputs(fplan)
        fsteps = 2
        fms, _ = time_steps(lambda: B.run_forward_backward(fplan, ft, fout), fsteps, 3, None)
        fms /= fsteps
        rec.update({"flattened_ms_per_step": fms, "speedup_vs_flattened": fms / ms, "meets_reuse_factor": bool(fms / ms >= fl["reuse_factor"])})
        del fout, ft
    torch.cuda.empty_cache()
    return rec


def run_strong(args, B, base, rank, world, local_rank, dist, pk):
    """--scaling strong: ONE workload split over the ranks with no exchange step (whole groups, or (group, KV head)
    pairs when there are fewer groups than ranks: workloads.partition).  Every rank generates the same seeded tensors
    and keeps its parts' slices; `value` is the whole workload's useful FLOPs over the slowest rank's time."""
    fl = useful_flops(base)
    parts = wl.partition(base, world)[rank]
    big = (base.total_prompt + base.total_response) * base.h_q * base.head_dim > 2e8
    full = {k: v.cuda() for k, v in wl.make_tensors(base, device="cuda" if big else "cpu").items()}
    jobs = []
    for part in parts:
        pw = wl.part_workload(base, part)
        pt = wl.part_tensors(base, full, part)
        plan = B.Plan(pw.prompt_len, pw.branch_len, pw.h_q, pw.h_kv, pw.head_dim, device=local_rank, flags=B.FLAG_ZERO_PROMPT_GRAD,
                      kv_splits=4 if pw.extra.get("force_split") else 0)
        jobs.append((pw, plan, pt, B.alloc_outputs(plan)))
    del full

    def step():
        for _, plan, pt, out in jobs:
            B.run_forward_backward(plan, pt, out)

    l0 = B.launch_count()
    ms, clocks = time_steps(step, args.steps, args.warmup, dist, sampler_index=local_rank if rank == 0 else None)
    launches = (B.launch_count() - l0) // (args.steps + args.warmup) * args.steps
    for _, plan, _, _ in jobs:
        if plan.device_status() != (0, 0):
            raise RuntimeError("device status")
    ms_step = ms / args.steps
    mine = sum(useful_flops(pw)["total"] for pw, _, _, _ in jobs)
    if rank == 0:
        value = fl["total"] / (ms_step * 1e-3) / 1e12
        line = {"metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic", "config": {**config_record(base, 1), "parallelism": f"one workload over {world} ranks: "
                                                "whole groups or (group, KV head) units, no exchange step"},
                "rank0_share_of_flops": mine / fl["total"], "rank0_parts": [[p.groups, p.kv_heads] for p in parts],
                "pct_of_measured_bf16_peak": 100 * value / world / pk["bf16_tflops"], "gpu_launches": int(launches), "clocks": clocks,
                "e2e": None, "roofline": None, "cpu_baseline": None}
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload configuration 1..5 (default 2, the metric's)")
    ap.add_argument("--no-flattened", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-configs", action="store_true", help="skip the brief runs of the other four configurations")
    ap.add_argument("--scale-down", type=int, default=1,
                    help="divide every length of the configuration by this (small cases of the same kernels for ncu captures; "
                         "the workload's name in `config` carries the divisor)")
    ap.add_argument("--e2e-chunks", type=int, default=4,
                    help="runs of branches the host-buffer leg cuts the replay calls into (1: the four calls as they are)")
    ap.add_argument("--bwd-handoff", action="store_true",
                    help="backward calls take the dS hand-off path (5 GEMMs per tile pair, 32 KB of scratch per pair and head)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak (default): every rank runs its own groups; strong: one workload partitioned over the ranks")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = wl.config(args.config, args.scale_down)
    if args.scale_down != 1:
        w.name = f"{w.name}/{args.scale_down}"

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, w)
        return 0

    from paper_2609_33133_b200 import build
    build.build()
    from paper_2609_33133_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod
    pk = peaks()
    if args.scaling == "strong":
        run_strong(args, B, w, rank, world, local_rank, dist, pk)
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return 0
    w = rank_workload(w, rank)
    fl = useful_flops(w)

    big = (w.total_prompt + w.total_response) * w.h_q * w.head_dim > 2e8
    t_dev = wl.make_tensors(w, device="cuda" if big else "cpu")
    t_dev = {k: v.cuda() for k, v in t_dev.items()}
    splits = 4 if w.extra.get("force_split") else 0
    t_plan = time.perf_counter()
    plan = B.Plan(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim, device=local_rank, flags=B.FLAG_ZERO_PROMPT_GRAD,
                  kv_splits=splits)
    plan_ms = (time.perf_counter() - t_plan) * 1e3  # pack and schedule on the host + table upload; not part of a step
    out = B.alloc_outputs(plan, handoff_limit=(1 << 62) if args.bwd_handoff else 0)
    handoff = out["ws"].numel() >= plan.ws_bwd_handoff_bytes
    out_ws_bytes = out["ws"].numel()

    def step():
        B.run_forward_backward(plan, t_dev, out)

    # ---- main timed region (inputs resident in HBM), with per-kernel events for the roofline
    plan.set_timing(True)
    l0 = B.launch_count()
    ms, clocks = time_steps(step, args.steps, args.warmup, dist, sampler_index=local_rank if rank == 0 else None)
    launches = (B.launch_count() - l0) // (args.steps + args.warmup) * args.steps
    st = plan.device_status()
    if st != (0, 0):
        raise RuntimeError(f"device status {st}")
    kt = [plan.kernel_time(k) for k in range(6)]
    plan.set_timing(False)
    ms_step = ms / args.steps
    per_step = sorted(time_steps.per_step)
    value = aggregate_tflops(fl["total"], world, ms_step)

    # dominant kernel: the replay backward tile kernel
    names = ["prefill_fwd", "replay_fwd", "replay_bwd_dkdv", "prefill_bwd_dkdv", "replay_bwd_dq", "prefill_bwd_dq"]
    kfun = {"prefill_fwd": "fwd_kernel", "replay_fwd": "fwd_kernel", "replay_bwd_dkdv": "bwd_kernel", "prefill_bwd_dkdv": "bwd_kernel",
            "replay_bwd_dq": "dql_kernel" if handoff else "dq_kernel", "prefill_bwd_dq": "dql_kernel" if handoff else "dq_kernel"}
    per_kernel = {}
    for n, (tot, cnt) in zip(names, kt):
        if cnt:
            # tflops: the GEMM FLOPs the launch executes; tflops_algorithmic: its share of the 14 d per pair (the
            # query-side kernel's S and dP are recomputation: only its dQ GEMM, 2 d of its 6 d, is algorithmic)
            alg = fl[n] / 3 if n.endswith("_dq") else fl[n]
            executed = alg if handoff else fl[n]     # on the hand-off path the query-side launch is the dQ GEMM alone
            per_kernel[n] = {"ms": tot / cnt, "tflops": executed / (tot / cnt * 1e-3) / 1e12,
                             "tflops_algorithmic": alg / (tot / cnt * 1e-3) / 1e12, "launches": cnt}
    dom = max(per_kernel, key=lambda n: per_kernel[n]["ms"])
    roofline = {"bound": "tensor", "kernel": f"{kfun[dom]} ({dom})", "achieved": per_kernel[dom]["tflops"],
                "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": per_kernel[dom]["tflops"] / pk["bf16_tflops"],
                "peak_source": f"{pk['source']} cuBLAS bf16 burst", "traffic": ncu_dram_bytes(w.name, dom),
                "algorithmic_bytes": algorithmic_bytes(w, dom),
                # the kernel is timed inside a loop of steps that runs under the power cap; against the sustained figure:
                "peak_sustained": pk["bf16_tflops_sustained"], "frac_sustained": per_kernel[dom]["tflops"] / pk["bf16_tflops_sustained"]}

    # ---- end to end: pinned host inputs copied in, results copied out, every step
    host_in = {k: v.cpu().pin_memory() for k, v in t_dev.items()}
    res_names = ["o_p", "lse_p", "o_r", "lse_r", "dq_p", "dq_r", "dk_r", "dv_r", "dk_p", "dv_p"]
    host_out = {k: torch.empty(out[k].shape, dtype=out[k].dtype).pin_memory() for k in res_names}
    h2d = sum(v.numel() * v.element_size() for v in host_in.values())
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())

    # copies overlapped with the calls as far as the data flow allows; the replay calls run in runs of branches so that a
    # run's results leave, and the next run's inputs arrive, under the kernels
    host_step = B.HostStep(plan, t_dev, out, chunks=args.e2e_chunks)

    def step_e2e():
        host_step.run(host_in, host_out)

    e2e = None
    if not args.no_e2e:
        ms_e2e, _ = time_steps(step_e2e, max(3, args.steps // 2), 3, dist)
        ms_e2e /= max(3, args.steps // 2)
        e2e = {"value": aggregate_tflops(fl["total"], world, ms_e2e), "unit": "TFLOP/s", "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "replay_runs": len(host_step.runs) or 1}

    # ---- flattened no-reuse baseline: same kernels, prompt duplicated per branch
    flat = None
    if not args.no_flattened and rank == 0:
        del host_in, host_out
        fw = w.flattened()
        ft = wl.flatten_tensors(w, {k: v for k, v in t_dev.items()})
        e = lambda h: torch.empty((0, h, w.head_dim), dtype=torch.bfloat16, device="cuda")
        ft.update({"q_r": e(w.h_q), "k_r": e(w.h_kv), "v_r": e(w.h_kv), "do_r": e(w.h_q)})
        fplan = B.Plan(fw.prompt_len, fw.branch_len, fw.h_q, fw.h_kv, fw.head_dim, device=local_rank, flags=B.FLAG_ZERO_PROMPT_GRAD)
        fout = B.alloc_outputs(fplan)
        fsteps = max(3, args.steps // 4)
        fms, _ = time_steps(lambda: B.run_forward_backward(fplan, ft, fout), fsteps, 3, None)
        fms /= fsteps
        flat = {"ms_per_step": fms, "speedup": fms / ms_step, "reuse_factor": fl["reuse_factor"],
                "tflops_executed": fl["flattened_total"] / (fms * 1e-3) / 1e12}
        del fout, ft

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        info = oracle_sample(w, seconds_budget=15.0)
        cpu = {"value": fl["total"] / info["est_total_s"] / 1e12, "unit": "TFLOP/s", "cores": info["cores"], "kind": "oracle",
               "sample": f"{info['sequences']} of {info['of']} flattened (branch, head) sequences, {info['seconds_sample']:.1f} s, extrapolated"}

    # ---- the other four configurations, briefly (3 timed steps each; `value` stays the default workload's)
    others = None
    if rank == 0 and world == 1 and args.config == 2 and args.scale_down == 1 and not args.no_configs:
        del out, t_dev
        torch.cuda.empty_cache()
        others = {}
        for index in (1, 3, 4, 5):
            try:
                others[f"cfg{index}"] = measure_config(B, index, local_rank)
            except (RuntimeError, torch.OutOfMemoryError) as exc:   # reported, not fatal: the headline line still prints
                others[f"cfg{index}"] = {"error": str(exc)[:200]}
                torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": per_step[0],
            "plan_create_ms": plan_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": config_record(w, world),
            "pct_of_measured_bf16_peak": 100 * value / world / pk["bf16_tflops"],
            "pct_of_measured_bf16_sustained": 100 * value / world / pk["bf16_tflops_sustained"],
            "pct_of_nominal_bf16_peak": 100 * value / world / NOMINAL_BF16_TFLOPS,
            "kernels": per_kernel, "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "flattened": flat, "cpu_baseline": cpu, "configs": others,
            "bwd_path": "dS hand-off (5 GEMMs per tile pair)" if handoff else "recompute (7 GEMMs per tile pair)",
            "bwd_scratch_bytes": int(out_ws_bytes),
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
