"""The N > 1 path of the benchmark on CPU: two gloo ranks (no GPU, no data-path collective).

Ranks replay independent groups, so the only cross-rank steps are the barrier and the max over ranks of
the timed region; this checks the sharding rule and that reduction with world_size 2 over 127.0.0.1.
"""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2609_33133_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.rank_workload(wl.config(1), rank)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, dist, device="cpu")
    val = bench.aggregate_tflops(bench.useful_flops(w)["total"], world, ms)
    out.put((rank, w.seed, w.prompt_len, ms, val))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    base = wl.config(1)
    assert [r[1] for r in res] == [base.seed, base.seed + 1]          # own trees per rank ...
    assert all(r[2] == base.prompt_len for r in res)                  # ... of the same shape (weak scaling)
    assert all(abs(r[3] - 15.0) < 1e-9 for r in res)                  # max over ranks
    fl = bench.useful_flops(base)["total"]
    assert all(abs(r[4] - 2 * fl / 15e-3 / 1e12) < 1e-9 for r in res)  # whole-job value over the slowest rank's time


def _partition_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    res = {}
    for index in (1, 2, 3, 5):
        w = wl.config(index)
        mine = wl.partition(w, world)[rank]
        units = [(g, c) for part in mine for g in part.groups for c in part.kv_heads]
        flops = sum(bench.useful_flops(wl.part_workload(w, part))["total"] for part in mine)
        gathered = [None] * world
        dist.all_gather_object(gathered, (units, flops))          # the only cross-rank step: bookkeeping, not data
        res[index] = gathered
    out.put((rank, res))
    dist.barrier()
    dist.destroy_process_group()


def test_partition_covers_every_group_and_kv_head_once_on_two_ranks():
    """Strong-scaling shards (whole groups, or (group, KV head) units when groups < ranks): every unit on exactly one
    rank, the ranks' useful FLOPs add up to the workload's, and both ranks see the same answer."""
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_partition_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1]
    for index, gathered in res[0].items():
        w = wl.config(index)
        units = [u for us, _ in gathered for u in us]
        assert sorted(units) == [(g, c) for g in range(w.n_groups) for c in range(w.h_kv)], index
        assert sum(f for _, f in gathered) == bench.useful_flops(w)["total"], index
        loads = [f for _, f in gathered]
        assert max(loads) <= 0.56 * sum(loads), (index, loads)     # largest-first keeps two ranks within a few percent
    # fewer units than ranks: the extra ranks get nothing, nothing is lost
    w = wl.config(2)
    shards = wl.partition(w, 8)
    assert sum(len(s) for s in shards) == 4 and sum(1 for s in shards if not s) == 4


def test_flop_accounting_matches_oracle_pair_count():
    from oracle import tree_attention as ora
    for i in (1, 2, 3):
        w = wl.config(i)
        pre, rep, flat = ora.valid_pairs(ora.TreeBatch(w.prompt_len, w.branch_len, w.h_q, w.h_kv, w.head_dim))
        fl = bench.useful_flops(w)
        assert fl["total"] == 14 * w.head_dim * w.h_q * (pre + rep)
        assert abs(fl["reuse_factor"] - flat / (pre + rep)) < 1e-12
    assert abs(bench.useful_flops(wl.config(2))["total"] / 1e12 - 9.2606) < 1e-3


def test_bench_records_are_consistent():
    """Both arms print the same `config` object; the algorithmic bytes of the dominant launch are the sum of the tensors
    it touches, each crossing once; the tracked ncu table, where present, names the six launches of a step."""
    import json
    import os
    w = wl.config(2)
    assert bench.config_record(w, 1) == bench.config_record(wl.config(2), 1)
    # replay key-side backward on configuration 2: Q_R + dO_R 235 MB, statistics 3.7, K/V_R 33.6, K/V_P 16.8, dK_R/dV_R 33.6,
    # fp32 dK_P/dV_P read + written 67.1
    q, kv_r, kv_p = 2 * 16384 * 28 * 128, 2 * 16384 * 4 * 128, 2 * 8192 * 4 * 128
    want = 2 * q + 8 * 16384 * 28 + 2 * kv_r + 2 * kv_p + 2 * kv_r + 2 * 2 * (2 * kv_p)
    assert bench.algorithmic_bytes(w, "replay_bwd_dkdv") == want and abs(want / 1e9 - 0.39) < 0.005
    path = os.path.join(os.path.dirname(os.path.abspath(bench.__file__)), "profiles", "ncu_dram_bytes.json")
    if os.path.exists(path):
        table = json.load(open(path))
        for name, rec in table.items():
            if not name.startswith("_"):
                assert sorted(rec) == sorted(["prefill_fwd", "replay_fwd", "replay_bwd_dkdv", "replay_bwd_dq", "prefill_bwd_dkdv", "prefill_bwd_dq"])
                assert bench.ncu_dram_bytes(name, "replay_bwd_dkdv") == rec["replay_bwd_dkdv"] > bench.algorithmic_bytes(wl.config(2), "replay_bwd_dkdv") * 0.5
