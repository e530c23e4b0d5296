"""Turn Nsight Compute output into the short text summaries kept under profiles/.

  python -m paper_1805_07941_b200.profile_summary launches <ncu --csv log> [--title T] [--command C]
      per kernel: launches, total device time, share (from a `--metrics gpu__time_duration.sum` run)
  python -m paper_1805_07941_b200.profile_summary traffic <ncu --csv log> --last N [--first I] [--kernel REGEX]
      DRAM bytes (read + write) and time of N launches of the matching kernels (from launch I, else the
      last N), per launch
  python -m paper_1805_07941_b200.profile_summary counters <ncu --page raw --csv export> [--kernel REGEX]
      the handful of counters the roofline discussion uses, for each captured launch

It only parses text; nothing here touches a GPU.
"""
import argparse
import collections
import csv
import hashlib
import os
import re
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))

COUNTERS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed",
    "sm__inst_executed.avg.per_cycle_active", "sm__warps_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_alu_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_fma_cycles_active.avg.pct_of_peak_sustained_active",
    "launch__registers_per_thread", "launch__grid_size", "launch__block_size",
    "launch__occupancy_limit_registers", "launch__occupancy_limit_shared_mem",
    "lts__t_sector_hit_rate.pct", "l1tex__t_sector_hit_rate.pct",
    "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_not_selected_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_no_instruction_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_sleeping_per_issue_active.ratio",
]


def csrc_sha256():
    """Fingerprint of the CUDA sources: a stored traffic figure is valid only for the kernels it was taken on."""
    h = hashlib.sha256()
    d = os.path.join(_HERE, "csrc")
    for f in sorted(os.listdir(d)):
        if f.endswith((".cu", ".cuh")):
            with open(os.path.join(d, f), "rb") as fh:
                h.update(fh.read())
    return h.hexdigest()


def _rows(path):
    with open(path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    return list(csv.reader(lines))


def _to_us(value, unit):
    v = float(value.replace(",", ""))
    return {"ns": v / 1e3, "us": v, "ms": v * 1e3, "s": v * 1e6}.get(unit, v)


def _to_bytes(value, unit):
    v = float(value.replace(",", ""))
    return v * {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}.get(unit, 1)


def _short(name):
    name = re.sub(r"\(.*", "", name)
    return name.replace("void ", "").strip()


def launches(args):
    rows = _rows(args.file)
    hdr = rows[0]
    ki, mi, vi, ui = (hdr.index(c) for c in ("Kernel Name", "Metric Name", "Metric Value", "Metric Unit"))
    agg = collections.OrderedDict()
    for r in rows[1:]:
        if r[mi] != "gpu__time_duration.sum":
            continue
        a = agg.setdefault(_short(r[ki]), [0, 0.0])
        a[0] += 1
        a[1] += _to_us(r[vi], r[ui])
    total = sum(a[1] for a in agg.values())
    print("# %s" % (args.title or "kernel launch list"))
    if args.command:
        print("\ncommand: `%s`\n" % args.command)
    print("Device time per launch under ncu is cold-cache and serialised: compare shares, not absolutes.\n")
    print("| kernel | launches | total us | share | avg us |\n|---|---|---|---|---|")
    for n, a in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        print("| `%s` | %d | %.1f | %.1f%% | %.1f |" % (n, a[0], a[1], 100 * a[1] / total, a[1] / a[0]))


def traffic(args):
    rows = _rows(args.file)
    hdr = rows[0]
    ii, ki, mi, vi, ui = (hdr.index(c) for c in ("ID", "Kernel Name", "Metric Name", "Metric Value", "Metric Unit"))
    per = collections.OrderedDict()
    for r in rows[1:]:
        if not re.search(args.kernel, r[ki]):
            continue
        d = per.setdefault(r[ii], {"name": _short(r[ki])})
        if r[mi] == "gpu__time_duration.sum":
            d["us"] = _to_us(r[vi], r[ui])
        elif r[mi] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            d[r[mi]] = _to_bytes(r[vi], r[ui])
    allv = list(per.values())
    last = allv[args.first:args.first + args.last] if args.first >= 0 else allv[-args.last:]
    rd = sum(d.get("dram__bytes_read.sum", 0) for d in last)
    wr = sum(d.get("dram__bytes_write.sum", 0) for d in last)
    us = sum(d.get("us", 0) for d in last)
    print("# %s" % (args.title or "DRAM traffic"))
    if args.command:
        print("\ncommand: `%s`\n" % args.command)
    if args.first >= 0:
        print("Launches %d..%d of the %d matching `%s` (one pass over the workload, launched one by one):\n"
              % (args.first + 1, args.first + len(last), len(allv), args.kernel))
    else:
        print("Last %d launches matching `%s` (one pass over the workload, launched one by one):\n" % (len(last), args.kernel))
    print("- dram read: %.1f MB, dram write: %.1f MB, device time under ncu: %.1f us" % (rd / 1e6, wr / 1e6, us))
    print("- traffic_bytes_per_launch: %d" % round((rd + wr) / max(1, len(last))))
    print("- launches: %d" % len(last))
    print("- csrc_sha256: %s" % csrc_sha256())


def counters(args):
    with open(args.file, newline="") as f:
        rows = list(csv.reader(f))
    hdr, units = rows[0], rows[1]
    ki = hdr.index("Kernel Name")
    print("# %s" % (args.title or "ncu counters"))
    if args.command:
        print("\ncommand: `%s`\n" % args.command)
    for r in rows[2:]:
        if not re.search(args.kernel, r[ki]):
            continue
        print("## `%s`\n" % _short(r[ki]))
        for c in COUNTERS:
            if c in hdr:
                print("- %s: %s %s" % (c, r[hdr.index(c)], units[hdr.index(c)]))
        print()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("mode", choices=["launches", "traffic", "counters", "sha"])
    ap.add_argument("file", nargs="?")
    ap.add_argument("--title")
    ap.add_argument("--command")
    ap.add_argument("--kernel", default=".")
    ap.add_argument("--last", type=int, default=53, help="how many launches to sum")
    ap.add_argument("--first", type=int, default=-1, help="0-based index of the first launch (default: the last ones)")
    args = ap.parse_args()
    if args.mode == "sha":
        print(csrc_sha256())
        return
    {"launches": launches, "traffic": traffic, "counters": counters}[args.mode](args)


if __name__ == "__main__":
    main()
