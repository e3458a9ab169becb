#!/usr/bin/env python
"""Writes profiles/ncu_dram_bytes.json, the DRAM traffic per launch that bench.py reports as `roofline.traffic`.

Input: the raw-page CSV of an ncu capture of bench.py (tile kernels only, whole steps), e.g.

    CMD="python bench.py --steps 2 --warmup 3 --no-flattened --no-cpu-baseline --no-e2e --no-configs"
    $CMD && ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none \\
        -k regex:"fwd_kernel|bwd_kernel|dq_kernel" -s 6 -c 6 -f -o prof_dram $CMD
    ncu -i prof_dram.ncu-rep --page raw --csv > prof_dram.csv
    python bench_ncu_bytes.py prof_dram.csv cfg2-7b-layer "<the ncu command>"

One step launches, in order: fwd_kernel (prefill), fwd_kernel (replay), bwd_kernel (replay), dq_kernel (replay),
bwd_kernel (prefill), dq_kernel (prefill); the capture must start at a step boundary.
"""
import csv
import json
import os
import sys

ORDER = ["prefill_fwd", "replay_fwd", "replay_bwd_dkdv", "replay_bwd_dq", "prefill_bwd_dkdv", "prefill_bwd_dq"]
EXPECT = ["fwd_kernel", "fwd_kernel", "bwd_kernel", "dq_kernel", "bwd_kernel", "dq_kernel"]
UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def main():
    path, workload, command = sys.argv[1], sys.argv[2], sys.argv[3]
    rows = list(csv.reader(open(path)))
    hdr, units, data = rows[0], rows[1], rows[2:]
    name, rd, wr = hdr.index("Kernel Name"), hdr.index("dram__bytes_read.sum"), hdr.index("dram__bytes_write.sum")
    assert len(data) >= 6, "need one whole step (6 tile-kernel launches)"
    out = {}
    for k, exp, row in zip(ORDER, EXPECT, data[:6]):
        assert exp in row[name], (k, row[name])
        out[k] = float(row[rd].replace(",", "")) * UNIT[units[rd]] + float(row[wr].replace(",", "")) * UNIT[units[wr]]
    dst = os.path.join(os.path.dirname(os.path.abspath(__file__)), "profiles", "ncu_dram_bytes.json")
    table = json.load(open(dst)) if os.path.exists(dst) else {}
    table[workload] = out
    table.setdefault("_commands", {})[workload] = command
    json.dump(table, open(dst, "w"), indent=1, sort_keys=True)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
