"""Measurement plumbing: turns an ncu report into the short tables kept under profiles/ and into the DRAM-traffic
records bench.py reports (profiles/traffic.json).  Runs where the report is read, without a GPU.

  python -m paper_2601_13155_b200.ncu_summary REPORT.ncu-rep [extra metric names ...]
      prints one line per captured launch: duration, DRAM bytes read / written, DRAM and tensor-pipe utilisation,
      registers per thread.

  python -m paper_2601_13155_b200.ncu_summary --launch-list LAUNCHES.csv
      the launch list of a whole run (the CSV log of `ncu --metrics gpu__time_duration.sum --csv --log-file ...`):
      launches, total time and share per kernel.

  python -m paper_2601_13155_b200.ncu_summary REPORT.ncu-rep --traffic OP=KERNEL_REGEX[@INDEX] ... \
         --workload cfg3 --shape "m_ffn = 13108" --command "<the command that was profiled>"
      additionally records, for every OP given, dram__bytes_read.sum + dram__bytes_write.sum of the INDEX-th (default
      first) captured launch whose kernel name matches, in profiles/traffic.json, together with the SHA-256 of the
      source files the kernel is built from.  bench.py reports a record's traffic only while those files are unchanged.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import io
import json
import os
import re
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "traffic.json")

# source files whose change invalidates a captured traffic figure, per operation tag
OP_SOURCES = {
    "gate_up": ["csrc/kernels_tc_gemm.cu", "csrc/tc_ptx.cuh"],
    "down": ["csrc/kernels_tc_gemm.cu", "csrc/tc_ptx.cuh"],
    "qv_proj": ["csrc/kernels_tc_gemm.cu", "csrc/tc_ptx.cuh"],
    "o_proj": ["csrc/kernels_tc_gemm.cu", "csrc/tc_ptx.cuh"],
    "kproj_pap": ["csrc/kernels_tc_gemm.cu", "csrc/tc_ptx.cuh"],
    "attention": ["csrc/kernels_tc_attn.cu", "csrc/tc_ptx.cuh"],
    "decode": ["csrc/kernels_decode.cu"],
}


def source_digest(op: str) -> str:
    h = hashlib.sha256()
    for rel in OP_SOURCES[op]:
        with open(os.path.join(PKG, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def load_traffic() -> dict:
    if not os.path.exists(TRAFFIC_JSON):
        return {"records": []}
    with open(TRAFFIC_JSON) as f:
        return json.load(f)


def traffic_for(workload: str, op: str):
    """The captured DRAM bytes per launch of `op` at `workload`'s first-stage shape, or None when there is no record
    or the kernel's sources have changed since the capture."""
    if op not in OP_SOURCES:
        return None
    for r in load_traffic()["records"]:
        if r["workload"] == workload and r["op"] == op:
            return r if r["source_sha256"] == source_digest(op) else None
    return None


def read_report(path):
    out = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True, text=True).stdout
    rows = list(csv.reader(io.StringIO(out)))
    hdr, units = rows[0], rows[1]
    col = {h: i for i, h in enumerate(hdr)}

    def num(x):
        try:
            return float(x.replace(",", ""))
        except Exception:
            return float("nan")

    def get(r, n, d=""):
        i = col.get(n)
        return r[i] if i is not None and i < len(r) else d

    def unit(n):
        return units[col[n]] if n in col else ""

    scale_b = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    scale_t = {"ns": 1e-3, "us": 1, "ms": 1e3, "s": 1e6}
    launches = []
    for r in rows[2:]:
        name = re.sub(r"\(.*$", "", get(r, "Kernel Name")).replace("void ", "").replace("spts::<unnamed>::", "")
        launches.append({
            "name": name, "grid": get(r, "Grid Size"),
            "us": num(get(r, "gpu__time_duration.sum")) * scale_t.get(unit("gpu__time_duration.sum"), 1),
            "read": num(get(r, "dram__bytes_read.sum")) * scale_b.get(unit("dram__bytes_read.sum"), 1),
            "write": num(get(r, "dram__bytes_write.sum")) * scale_b.get(unit("dram__bytes_write.sum"), 1),
            "dram_pct": num(get(r, "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "nan")),
            "tensor_pct": num(get(r, "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed", "nan")),
            "regs": get(r, "launch__registers_per_thread"), "raw": r, "get": lambda n, r=r: get(r, n)})
    return launches


def launch_list(path):
    import collections
    lines = [l for l in open(path) if l.startswith('"')]
    agg = collections.OrderedDict()
    for row in csv.DictReader(lines):
        short = re.sub(r"^void ", "", row["Kernel Name"])
        short = re.sub(r"spts::<unnamed>::", "", short)
        short = re.sub(r"\(.*$", "", short)
        if len(short) > 70:
            short = short[:67] + "..."
        a = agg.setdefault(short, [0, 0.0])
        a[0] += 1
        a[1] += float(row["Metric Value"].replace(",", ""))
    tot = sum(v[1] for v in agg.values())
    mine = {k: v for k, v in agg.items() if not k.startswith("at::") and "elementwise" not in k}
    tm = sum(v[1] for v in mine.values())
    print(f"all kernels: {sum(v[0] for v in agg.values())} launches, {tot / 1e6:.1f} ms; library kernels: "
          f"{sum(v[0] for v in mine.values())} launches, {tm / 1e6:.1f} ms")
    print(f"{'kernel':70s} {'launches':>8s} {'total ms':>10s} {'avg us':>9s} {'share':>7s}")
    for k, v in sorted(mine.items(), key=lambda kv: -kv[1][1]):
        print(f"{k:70s} {v[0]:8d} {v[1] / 1e6:10.3f} {v[1] / v[0] / 1e3:9.1f} {100 * v[1] / tm:6.2f}%")


def main():
    if len(sys.argv) == 3 and sys.argv[1] == "--launch-list":
        return launch_list(sys.argv[2])
    ap = argparse.ArgumentParser()
    ap.add_argument("report")
    ap.add_argument("extra", nargs="*", help="further metric names to print")
    ap.add_argument("--traffic", nargs="*", default=[], metavar="OP=REGEX[@INDEX]")
    ap.add_argument("--decode-rows", type=int, default=0, metavar="CACHED_ROWS",
                    help="the report holds decode kernels against caches of this many rows: record the bytes one layer's "
                         "weight-streaming kernels move and the bytes per cached row of the attention kernel (op 'decode')")
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--shape", default="")
    ap.add_argument("--command", default="")
    a = ap.parse_args()
    launches = read_report(a.report)
    print(f"{'kernel':40s} {'grid':>14s} {'us':>8s} {'dramR MB':>9s} {'dramW MB':>9s} {'GB/s':>7s} {'dram%':>6s} {'tensor%':>7s} "
          f"{'regs':>4s}" + "".join(f" {e[-28:]:>28s}" for e in a.extra))
    for l in launches:
        print(f"{l['name'][:40]:40s} {l['grid']:>14s} {l['us']:8.1f} {l['read'] / 1e6:9.2f} {l['write'] / 1e6:9.2f} "
              f"{(l['read'] + l['write']) / l['us'] / 1e3:7.0f} {l['dram_pct']:6.1f} {l['tensor_pct']:7.1f} {l['regs']:>4s}"
              + "".join(f" {l['get'](e):>28s}" for e in a.extra))
    if a.decode_rows:
        first = next(i for i, l in enumerate(launches) if "dec_qkv_kernel" in l["name"])
        second = next(i for i, l in enumerate(launches[first + 1:], first + 1) if "dec_qkv_kernel" in l["name"])
        layer = launches[first:second]
        attn = sum(l["read"] + l["write"] for l in layer if "dec_attn_mma" in l["name"] or "dec_attn_partial" in l["name"])
        rest = sum(l["read"] + l["write"] for l in layer) - attn
        try:
            commit = subprocess.run(["git", "-C", ROOT, "rev-parse", "--short", "HEAD"], capture_output=True, text=True).stdout.strip()
        except Exception:
            commit = ""
        rec = {"workload": "cfg5", "op": "decode", "kernel": "decode step, one layer", "shape": f"{a.decode_rows} cached rows per layer",
               "weight_bytes_per_layer": rest, "kv_bytes_per_row": attn / (a.decode_rows + 3.0),
               "dram_bytes_per_launch": rest + attn, "source_files": OP_SOURCES["decode"], "source_sha256": source_digest("decode"),
               "commit_at_capture": commit, "command": a.command}
        data = load_traffic()
        data["records"] = [r for r in data["records"] if r["op"] != "decode"] + [rec]
        data["records"].sort(key=lambda r: (r["workload"], r["op"]))
        with open(TRAFFIC_JSON, "w") as f:
            json.dump(data, f, indent=1)
            f.write("\n")
        print(f"recorded decode: {rest / 1e6:.1f} MB per layer of weight-streaming kernels, {rec['kv_bytes_per_row']:.0f} B per cached row")
        return
    if not a.traffic:
        return
    try:
        commit = subprocess.run(["git", "-C", ROOT, "rev-parse", "--short", "HEAD"], capture_output=True, text=True).stdout.strip()
    except Exception:
        commit = ""
    data = load_traffic()
    for spec in a.traffic:
        op, rx = spec.split("=", 1)
        index = 0
        if "@" in rx:
            rx, idx = rx.rsplit("@", 1)
            index = int(idx)
        hits = [l for l in launches if re.search(rx, l["name"])]
        if len(hits) <= index:
            sys.exit(f"no launch {index} matching {rx!r} in the report")
        l = hits[index]
        rec = {"workload": a.workload, "op": op, "kernel": l["name"], "grid": l["grid"], "shape": a.shape,
               "dram_bytes_read": l["read"], "dram_bytes_write": l["write"], "dram_bytes_per_launch": l["read"] + l["write"],
               "duration_us_under_ncu": l["us"], "source_files": OP_SOURCES[op], "source_sha256": source_digest(op),
               "commit_at_capture": commit, "command": a.command}
        data["records"] = [r for r in data["records"] if not (r["workload"] == a.workload and r["op"] == op)] + [rec]
        print(f"recorded {op}: {rec['dram_bytes_per_launch'] / 1e6:.1f} MB per launch ({l['name']})")
    data["records"].sort(key=lambda r: (r["workload"], r["op"]))
    with open(TRAFFIC_JSON, "w") as f:
        json.dump(data, f, indent=1)
        f.write("\n")


if __name__ == "__main__":
    main()
