"""Turns Nsight Compute output of a bench.py run into the short text summaries kept under profiles/.

    python -m paper_2511_02017_b200.profiling launches <launches.csv> <out.txt> "<command that made it>"
    python -m paper_2511_02017_b200.profiling kernel   <report.ncu-rep> <out.txt> "<command that made it>"
    python -m paper_2511_02017_b200.profiling traffic  <dram.csv> <bench.json> <out.json> "<command>"

`launches`: per kernel its launches, total time and share (gpu__time_duration.sum, one line per launch in
the csv).  `kernel`: the counters the roofline discussion uses, per captured launch.  `traffic`: DRAM
bytes moved per algorithmic byte, per kernel class, from a run that captured dram__bytes_read.sum and
dram__bytes_write.sum for every launch and whose bench line carries the lifetime row counts.
Reads files only; needs no GPU (the `kernel` mode calls `ncu -i`).
"""
import collections
import csv
import json
import subprocess
import sys

KEEP = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "dram__cycles_active.avg.pct_of_peak_sustained_elapsed",
    "sm__warps_active.avg.pct_of_peak_sustained_active", "launch__registers_per_thread", "launch__grid_size",
    "launch__block_size", "launch__cluster_size", "smsp__inst_executed.sum", "smsp__issue_active.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_active", "sm__inst_executed_pipe_fma.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_alu.avg.pct_of_peak_sustained_active", "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "lts__t_sector_hit_rate.pct", "sm__cycles_active.avg", "sm__cycles_elapsed.max",
]


def _csv_rows(path):
    rows = [r for r in csv.reader(open(path)) if len(r) > 5]
    for i, r in enumerate(rows):
        if r[0] == "ID":
            return r, rows[i + 1:]
    raise SystemExit("no csv header in " + path)


def _short(name):
    return name.split("(")[0].replace("void ", "")


def launches(src, dst, cmd):
    hdr, data = _csv_rows(src)
    ki, vi, ui = hdr.index("Kernel Name"), hdr.index("Metric Value"), hdr.index("Metric Unit")
    agg = collections.OrderedDict()
    for r in data:
        v = float(r[vi].replace(",", "")) * {"ns": 1e-3, "us": 1.0, "ms": 1e3}.get(r[ui], 1.0)
        a = agg.setdefault(_short(r[ki]), [0, 0.0])
        a[0] += 1
        a[1] += v
    tot = sum(a[1] for a in agg.values())
    with open(dst, "w") as f:
        f.write("command: %s\n" % cmd)
        f.write("(every launch replayed alone with cold caches: compare shares, not absolute times)\n\n")
        f.write("%-34s %9s %12s %8s %10s\n" % ("kernel", "launches", "total us", "share", "avg us"))
        for k, a in agg.items():
            f.write("%-34s %9d %12.1f %7.1f%% %10.2f\n" % (k, a[0], a[1], 100 * a[1] / tot, a[1] / a[0]))


def kernel(src, dst, cmd):
    out = subprocess.run(["ncu", "-i", src, "--page", "raw", "--csv"], capture_output=True, text=True).stdout
    rows = list(csv.reader(out.splitlines()))
    hdr, units = rows[0], rows[1]
    with open(dst, "w") as f:
        f.write("command: %s\n" % cmd)
        for r in rows[2:]:
            f.write("\n%s  grid %s block %s\n" % (_short(r[hdr.index("Kernel Name")]), r[hdr.index("Grid Size")],
                                                 r[hdr.index("Block Size")]))
            for m in KEEP:
                if m in hdr:
                    f.write("  %-70s %18s %s\n" % (m, r[hdr.index(m)], units[hdr.index(m)]))
            st = [(hdr[i], float(r[i].replace(",", ""))) for i in range(len(hdr))
                  if hdr[i].startswith("smsp__average_warps_issue_stalled") and hdr[i].endswith("_per_issue_active.ratio") and r[i]]
            st.sort(key=lambda x: -x[1])
            f.write("  top stall reasons (warps per issue): " + ", ".join(
                "%s %.2f" % (n.replace("smsp__average_warps_issue_stalled_", "").replace("_per_issue_active.ratio", ""), v)
                for n, v in st[:5]) + "\n")


def traffic(src, bench_json, dst, cmd):
    hdr, data = _csv_rows(src)
    ki, vi, ui, mi = hdr.index("Kernel Name"), hdr.index("Metric Value"), hdr.index("Metric Unit"), hdr.index("Metric Name")
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    tot = collections.defaultdict(float)
    for r in data:
        if r[mi].startswith("dram__bytes_"):
            tot[_short(r[ki]).split("<")[0]] += float(r[vi].replace(",", "")) * scale.get(r[ui], 1.0)
    line = [json.loads(l) for l in open(bench_json) if l.startswith("{")][-1]
    rb, life = line["config"]["row_bytes"], line["rows_lifetime"]
    alg = {"k_draft_stream+k_draft_finish": life["draft"] * rb, "k_verify_walk": (life["target"] + life["residual"]) * rb}
    dram = {"k_draft_stream+k_draft_finish": tot["k_draft_stream"] + tot["k_draft_finish"], "k_verify_walk": tot["k_verify_walk"]}
    from bench import kernel_source_digest
    rec = {"command": cmd, "workload": line["config"]["workload"], "source_digest": kernel_source_digest(),
           "dram_bytes": dram, "algorithmic_bytes": alg,
           "dram_bytes_per_alg_byte": {k: dram[k] / alg[k] for k in alg if alg[k] > 0}}
    json.dump(rec, open(dst, "w"), indent=1)


if __name__ == "__main__":
    mode = sys.argv[1]
    {"launches": launches, "kernel": kernel, "traffic": traffic}[mode](*sys.argv[2:])
