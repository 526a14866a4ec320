"""Turns the raw counter page of an ncu capture into the short summaries kept under profiles/.

    ncu -i capture.ncu-rep --page raw --csv > raw.csv
    python -m paper_2503_14153_b200.ncu_summary raw.csv --out profiles/NAME --command "the full capture command" \
        [--traffic-kernel 'gemm_cluster<64,swiglu>' --match gemm_cluster --launch 1 --shape 4096 11008 64 \
         --sources paper_2503_14153_b200/csrc/gemm_cluster.cuh]

    ncu --metrics gpu__time_duration.sum ... --csv --log-file launches.csv <cmd>
    python -m paper_2503_14153_b200.ncu_summary launches.csv --launch-list --last-step-from medusa_act_tc \
        --out profiles/NAME --command "..."

Writes NAME.md (one row per captured launch: duration, DRAM bytes, DRAM and tensor-pipe utilisation,
occupancy, registers) and, with --traffic-kernel, NAME.json holding the DRAM read + write bytes of
one launch together with a hash of the kernel's source files: the benchmark reports that figure as
`roofline.traffic` only while the hash still matches.
"""
import argparse
import csv
import hashlib
import json
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
COLS = [("gpu__time_duration.sum", "us"), ("dram__bytes_read.sum", "DRAM read MB"), ("dram__bytes_write.sum", "DRAM write MB"),
        ("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "DRAM %"),
        ("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active", "tensor pipe %"),
        ("sm__warps_active.avg.pct_of_peak_sustained_active", "warps active %"),
        ("launch__registers_per_thread", "regs"), ("lts__t_sector_hit_rate.pct", "L2 hit %"),
        ("lts__t_bytes.sum", "L2 MB")]


def to_number(value: str, unit: str):
    v = float(value.replace(",", ""))
    scale = {"ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6, "byte": 1e-6, "Kbyte": 1e-3, "Mbyte": 1.0, "Gbyte": 1e3}
    return v * scale.get(unit, 1.0)


def parse(path):
    """-> list of launches: {"name", "grid", "block", metric: value (us / MB / % / count)}"""
    lines = [l for l in open(path) if not l.startswith("==")]
    rows = list(csv.reader(lines))
    header, units, body = rows[0], rows[1], rows[2:]
    idx = {h: i for i, h in enumerate(header)}
    out = []
    for r in body:
        if len(r) < len(header):
            continue
        rec = {"name": re.sub(r"^void\s+", "", re.sub(r"\(.*", "", r[idx["Kernel Name"]])).replace("spec::", ""),
               "grid": r[idx["Grid Size"]], "block": r[idx["Block Size"]]}
        for m, _ in COLS:
            if m in idx and r[idx[m]] not in ("", "n/a"):
                rec[m] = to_number(r[idx[m]], units[idx[m]])
        out.append(rec)
    return out


def launch_list(path, last_step_from):
    """Per-kernel launches, total time and share of the launch list's last decode step (from the launch before
    the last `last_step_from` kernel on) out of a `--metrics gpu__time_duration.sum --csv` log."""
    lines = [l for l in open(path) if not l.startswith("==")]
    seq = []
    for row in csv.DictReader(lines):
        if row.get("Metric Name") != "gpu__time_duration.sum":
            continue
        name = re.sub(r"^void\s+", "", re.sub(r"\(.*", "", row["Kernel Name"])).replace("spec::", "")
        seq.append((name, to_number(row["Metric Value"], row["Metric Unit"]), row["Grid Size"]))
    if last_step_from:
        idx = [i for i, s in enumerate(seq) if last_step_from in s[0]]
        if idx:
            seq = seq[max(idx[-1] - 1, 0):]
    agg = {}
    for n, v, g in seq:
        a = agg.setdefault(f"{n} {g}", [0, 0.0])
        a[0] += 1
        a[1] += v
    return seq, agg


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--launch-list", action="store_true", help="the input is a gpu__time_duration launch list")
    ap.add_argument("--last-step-from", default=None, help="keep the launches from the one before the last kernel of this name")
    ap.add_argument("raw_csv")
    ap.add_argument("--out", required=True, help="path prefix of the .md (and .json) to write")
    ap.add_argument("--command", required=True, help="the full command that made the capture")
    ap.add_argument("--title", default=None)
    ap.add_argument("--traffic-kernel", default=None, help="name the benchmark knows the dominant kernel by")
    ap.add_argument("--match", default=None, help="substring of the captured kernel name to take the traffic from")
    ap.add_argument("--launch", type=int, default=0, help="which of the matching launches")
    ap.add_argument("--shape", type=int, nargs="+", default=None)
    ap.add_argument("--sources", nargs="+", default=[])
    args = ap.parse_args()
    if args.launch_list:
        seq, agg = launch_list(args.raw_csv, args.last_step_from)
        tot = sum(v for _, v, _ in seq)
        with open(args.out + ".md", "w") as f:
            f.write(f"# {args.title or os.path.basename(args.out)}\n\nCommand (B200, one GPU; the plain run exited 0 first):\n\n    {args.command}\n\n"
                    f"Launches of the last captured decode step ({len(seq)} launches, {tot:.1f} us in all; times under the profiler are "
                    "cold-cache and serialised: compare shares, not absolutes).\n\n")
            f.write("| kernel grid | launches | total us | share | avg us |\n|---|---|---|---|---|\n")
            for k, (c, t) in sorted(agg.items(), key=lambda x: -x[1][1]):
                f.write(f"| {k} | {c} | {t:.1f} | {t / tot * 100:.1f}% | {t / c:.2f} |\n")
        return
    launches = parse(args.raw_csv)
    with open(args.out + ".md", "w") as f:
        f.write(f"# {args.title or os.path.basename(args.out)}\n\nCommand (B200, one GPU; the plain run exited 0 first):\n\n    {args.command}\n\n")
        f.write("| # | kernel | grid | " + " | ".join(c for _, c in COLS) + " |\n|---|---|---|" + "---|" * len(COLS) + "\n")
        for i, l in enumerate(launches):
            f.write(f"| {i} | {l['name']} | {l['grid']} | " + " | ".join(f"{l[m]:.1f}" if m in l else "" for m, _ in COLS) + " |\n")
    if args.traffic_kernel:
        sel = [l for l in launches if args.match in l["name"]][args.launch]
        h = hashlib.sha256()
        for src in args.sources:
            h.update(open(os.path.join(ROOT, src), "rb").read())
        entry = {"kernel": args.traffic_kernel, "shape": args.shape, "captured_as": sel["name"], "grid": sel["grid"],
                 "dram_bytes_per_launch": (sel["dram__bytes_read.sum"] + sel["dram__bytes_write.sum"]) * 1e6,
                 "us_under_ncu": sel.get("gpu__time_duration.sum"), "sources": args.sources, "sources_sha16": h.hexdigest()[:16]}
        json.dump({"command": args.command, "kernels": [entry]}, open(args.out + ".json", "w"), indent=1)


if __name__ == "__main__":
    main()
