"""Turns Nsight Compute output into the short text summaries kept under profiles/.

    ncu -i capture.ncu-rep --page raw --csv > raw.csv
    python -m paper_2301_12187_b200.ncu_summary counters raw.csv --kernel k_conv_tc_rows --workload cfg4 \
        --source conv_tc_rows.cu
    python -m paper_2301_12187_b200.ncu_summary launches launches.csv

`counters` prints, per captured launch, the figures the roofline discussion uses (duration, DRAM
bytes and throughput, tensor-pipe activity, instruction and stall figures, launch shape) and one row
for profiles/dram_traffic.md: kernel | workload | DRAM bytes per launch | source file | first 16 hex
digits of the source file's SHA-256.  The benchmark reports that traffic only while the hash still
matches the kernel's source.  `launches` turns a `--metrics gpu__time_duration.sum --csv` log into a
per-kernel table of launches, total time and share.  Reads text files only; needs no GPU.
"""
from __future__ import annotations

import argparse
import collections
import csv
import hashlib
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))

COUNTERS = [
    ("gpu__time_duration.sum", "duration"),
    ("sm__cycles_elapsed.max", "SM cycles elapsed"),
    ("dram__bytes_read.sum", "DRAM bytes read"),
    ("dram__bytes_write.sum", "DRAM bytes written"),
    ("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "DRAM throughput, % of peak"),
    ("lts__t_sector_hit_rate.pct", "L2 sector hit rate, %"),
    ("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed", "tensor pipe active, % of elapsed"),
    ("sm__inst_executed.avg.per_cycle_elapsed", "warp instructions per cycle per SM"),
    ("smsp__inst_executed.sum", "warp instructions executed"),
    ("sm__warps_active.avg.per_cycle_active", "warps resident per SM (avg)"),
    ("launch__registers_per_thread", "registers per thread"),
    ("launch__grid_size", "grid size"),
    ("launch__block_size", "block size"),
    ("launch__shared_mem_per_block_dynamic", "dynamic shared memory per block"),
    ("l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum", "shared-memory bank conflicts"),
    ("smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio", "stall: long scoreboard (warps per issue)"),
    ("smsp__average_warps_issue_stalled_wait_per_issue_active.ratio", "stall: wait"),
    ("smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio", "stall: short scoreboard"),
    ("smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio", "stall: barrier"),
    ("smsp__average_warps_issue_stalled_no_instruction_per_issue_active.ratio", "stall: no instruction"),
    ("smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio", "stall: math pipe throttle"),
    ("smsp__average_warps_issue_stalled_lg_throttle_per_issue_active.ratio", "stall: LSU queue (lg throttle)"),
]

UNIT_BYTES = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def read_raw(path):
    """Rows of `ncu --page raw --csv`: header, units, then one row per captured launch."""
    with open(path, newline="") as f:
        rows = [r for r in csv.reader(l for l in f if l.startswith('"'))]
    if len(rows) < 3:
        raise SystemExit("no captured launches in %s" % path)
    return rows[0], rows[1], rows[2:]


def source_hash(name):
    path = os.path.join(HERE, "csrc", name)
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def counters(args):
    head, units, launches = read_raw(args.raw)
    col = {n: i for i, n in enumerate(head)}
    kcol = col.get("Kernel Name")
    for li, row in enumerate(launches):
        name = row[kcol].split("(")[0].replace("<unnamed>::", "").replace("void ", "") if kcol is not None else "?"
        if args.kernel and args.kernel not in name:
            continue
        print("### %s, launch %d of the capture" % (name, li))
        print()
        print("| counter | value |")
        print("|---|---|")
        traffic = 0.0
        for key, label in COUNTERS:
            if key not in col:
                continue
            val, unit = row[col[key]], units[col[key]]
            print("| %s (`%s`) | %s %s |" % (label, key, val, unit))
            if key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                traffic += float(val.replace(",", "")) * UNIT_BYTES.get(unit, 1.0)
        print()
        if args.source and args.workload:
            print("dram_traffic.md row:")
            print("| %s | %s | %d | %s | %s |" % (args.kernel or name, args.workload, round(traffic), args.source,
                                                  source_hash(args.source)))
            print()


def launches(args):
    for path in args.logs:
        with open(path, newline="") as f:
            rows = [r for r in csv.reader(l for l in f if l.startswith('"'))]
        h = rows[0]
        ik, iv, iu, im = h.index("Kernel Name"), h.index("Metric Value"), h.index("Metric Unit"), h.index("Metric Name")
        agg = collections.OrderedDict()
        for r in rows[1:]:
            if len(r) <= iv or r[im] != "gpu__time_duration.sum":
                continue
            v = float(r[iv].replace(",", ""))
            v = v / 1e3 if r[iu] == "ns" else (v * 1e3 if r[iu] == "ms" else v)
            name = r[ik].split("(")[0].replace("<unnamed>::", "").replace("void ", "")
            if "at::native" in name or "elementwise" in name:
                name = "torch kernels (buffers of the harness)"
            a = agg.setdefault(name, [0, 0.0])
            a[0] += 1
            a[1] += v
        total = sum(a[1] for a in agg.values())
        print("## %s: %d launches, %.1f us in total" % (os.path.basename(path), sum(a[0] for a in agg.values()), total))
        print()
        print("| kernel | launches | total us | avg us | share |")
        print("|---|---|---|---|---|")
        for k, (n, t) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
            print("| %s | %d | %.1f | %.2f | %.1f %% |" % (k, n, t, t / n, 100 * t / total))
        print()


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="cmd", required=True)
    c = sub.add_parser("counters")
    c.add_argument("raw")
    c.add_argument("--kernel", default="")
    c.add_argument("--workload", default="")
    c.add_argument("--source", default="", help="file under csrc/ that holds the kernel")
    c.set_defaults(fn=counters)
    l = sub.add_parser("launches")
    l.add_argument("logs", nargs="+")
    l.set_defaults(fn=launches)
    args = ap.parse_args(argv)
    args.fn(args)


if __name__ == "__main__":
    main(sys.argv[1:])
