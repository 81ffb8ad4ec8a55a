"""Turn an ncu metric capture of the hot loop into the DRAM-traffic record the benchmark reads.

    python -m paper_2608_15533_b200.ncu_traffic --csv CAPTURE.csv --config 1 --cap 16 \
        --command "<the ncu command line>" [--state fp32] [--out profiles/dram_traffic.json]

``CAPTURE.csv`` is what ``ncu --csv --log-file CAPTURE.csv --metrics
dram__bytes_read.sum,dram__bytes_write.sum ...`` wrote for a run of ``bench.py --only-hot-loop``.
Per kernel family (decode, merge, fused merge step, eager) the script records the number of
captured launches and the mean DRAM bytes read and written per launch.  The record is stamped
with the identifier of the library build it was captured on (``build.source_id()``: a hash of the
kernel sources and compiler switches); ``bench.py`` reports these figures only while the stamp
matches the library it is timing, and ``null`` otherwise.  A capture taken on another build
replaces the whole file (figures of different builds are never mixed).

Pure text processing: it needs neither a GPU nor the CUDA library.
"""
from __future__ import annotations

import argparse
import csv
import json
from pathlib import Path

from . import build

ROOT = Path(__file__).resolve().parent.parent
DEFAULT_OUT = ROOT / "profiles" / "dram_traffic.json"

_UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}
FAMILIES = (("fused_step_resident", "fused"), ("decode_merge_step", "fused"), ("decode_pipelined", "decode"), ("decode_append", "decode"),
            ("decode_multi", "decode_multi"), ("merge_tc", "merge"), ("merge_kernel", "merge"),
            ("eager_step", "eager"))


def family_of(kernel_name: str):
    for needle, fam in FAMILIES:
        if needle in kernel_name:
            return fam
    return None


def parse(csv_path: Path):
    """-> {launch id: {"kernel": name, "read": bytes, "write": bytes}} in launch order."""
    rows = [r for r in csv.reader(open(csv_path, newline="")) if len(r) > 8]
    hdr = next((r for r in rows if "Kernel Name" in r and "Metric Name" in r), None)
    if hdr is None:
        raise SystemExit(f"{csv_path}: no ncu CSV header found")
    col = {n: hdr.index(n) for n in ("ID", "Kernel Name", "Metric Name", "Metric Unit", "Metric Value")}
    launches = {}
    for r in rows[rows.index(hdr) + 1:]:
        try:
            lid = int(r[col["ID"]])
            value = float(r[col["Metric Value"]].replace(",", ""))
        except (ValueError, IndexError):
            continue
        metric, unit = r[col["Metric Name"]], r[col["Metric Unit"]]
        rec = launches.setdefault(lid, {"kernel": r[col["Kernel Name"]]})
        if metric == "dram__bytes_read.sum":
            rec["read"] = value * _UNIT.get(unit, 1.0)
        elif metric == "dram__bytes_write.sum":
            rec["write"] = value * _UNIT.get(unit, 1.0)
    return [launches[i] for i in sorted(launches) if "read" in launches[i] and "write" in launches[i]]


def summarise(launches):
    fams = {}
    for rec in launches:
        fam = family_of(rec["kernel"])
        if fam is None:
            continue
        f = fams.setdefault(fam, {"kernel": rec["kernel"].split("(")[0].replace("void deltalog::", ""),
                                  "launches": 0, "read": [], "write": []})
        f["launches"] += 1
        f["read"].append(rec["read"])
        f["write"].append(rec["write"])
    out = {}
    for fam, f in fams.items():
        n = f["launches"]
        out[fam] = {"kernel": f["kernel"], "launches": n,
                    "dram_read_bytes_per_launch": sum(f["read"]) / n,
                    "dram_write_bytes_per_launch": sum(f["write"]) / n,
                    "dram_read_bytes_min_max": [min(f["read"]), max(f["read"])]}
    return out


def capture_key(config: int, cap: int, state: str = "fp32") -> str:
    return f"config{config}_cap{cap}_{state}"


def load(path: Path = DEFAULT_OUT):
    try:
        return json.loads(Path(path).read_text())
    except (OSError, ValueError):
        return None


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--csv", required=True, type=Path)
    ap.add_argument("--config", required=True, type=int)
    ap.add_argument("--cap", required=True, type=int)
    ap.add_argument("--state", default="fp32")
    ap.add_argument("--command", required=True, help="the full ncu command line that produced the CSV")
    ap.add_argument("--build-id", default=None, help="identifier of the profiled build (default: the current sources)")
    ap.add_argument("--out", type=Path, default=DEFAULT_OUT)
    ap.add_argument("--add", action="store_true",
                    help="add the kernel families of this capture to the configuration's record instead of replacing it "
                         "(a second command of the same configuration, e.g. the eager kernel or the paper's cycle)")
    args = ap.parse_args(argv)

    build_id = args.build_id or build.source_id(build.extra_flags())
    kernels = summarise(parse(args.csv))
    if not kernels:
        raise SystemExit(f"{args.csv}: no launch of a library kernel with both DRAM counters")
    doc = load(args.out)
    if not doc or doc.get("build_id") != build_id:
        doc = {"build_id": build_id, "captures": {}}
    doc["what"] = ("dram__bytes_read.sum / dram__bytes_write.sum per launch (mean over the captured launches), "
                   "ncu --cache-control none: L2 as the previous launch of the loop left it")
    key = capture_key(args.config, args.cap, args.state)
    if args.add and key in doc["captures"]:
        rec = doc["captures"][key]
        rec["kernels"].update(kernels)
        rec.setdefault("more_commands", []).append(args.command)
    else:
        doc["captures"][key] = {"command": args.command, "kernels": kernels}
    args.out.write_text(json.dumps(doc, indent=1, sort_keys=True) + "\n")
    for fam, k in kernels.items():
        print(f"{fam:8s} {k['launches']:3d} launches  read {k['dram_read_bytes_per_launch'] / 1e6:8.1f} MB  "
              f"write {k['dram_write_bytes_per_launch'] / 1e6:7.1f} MB  {k['kernel'][:60]}")
    print(f"wrote {args.out} (build {build_id})")


if __name__ == "__main__":
    main()
