"""Turn an ncu capture of one of the FFN kernels into the record bench.py reads for its `traffic` figure.

    ncu -i capture.ncu-rep --page raw --csv > capture.csv          # on any machine with ncu
    python -m paper_2502_19078_b200.ncu_summary capture.csv --kernel sparse_ffn_kernel \
        --workload c2_llama2_7b_layer --units-per-launch 1 --note "40 % sparsity, launches of bench.py's FFN-only loop"

writes profiles/traffic_<kernel>.txt: the mean over the captured launches of dram__bytes_read.sum +
dram__bytes_write.sum, divided by the units (layer passes) one launch processes, together with a hash of the
kernel's source files.  bench.py reports the figure only while that hash still matches, so a record cannot
outlive the kernel it was taken from.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2502_19078_b200", "csrc")
KERNEL_SOURCES = {
    "sparse_ffn_kernel": ["clada_ffn.cu", "ffn_common.cuh", "common.cuh"],
    "sparse_ffn_stack_kernel": ["clada_ffn_stack.cu", "ffn_common.cuh", "common.cuh"],
    "sparse_ffn_batch_dense_kernel": ["clada_ffn_batch_dense.cu", "tc_common.cuh", "ffn_batch.cuh", "ffn_common.cuh",
                                      "common.cuh"],
    "sparse_ffn_batch_tc_kernel": ["clada_ffn_batch_tc.cu", "ffn_batch.cuh", "ffn_common.cuh", "common.cuh"],
}
_UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def sources_hash(kernel: str) -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def read_raw_csv(path: str, kernel: str):
    """Rows of `ncu --page raw --csv` whose kernel name contains `kernel`: list of {metric: value in base units}."""
    with open(path, newline="") as f:
        lines = [l for l in f if l.startswith('"')]
    rows = list(csv.reader(lines))
    header, units = rows[0], rows[1]
    out = []
    for row in rows[2:]:
        rec = dict(zip(header, row))
        if kernel not in rec.get("Kernel Name", ""):
            continue
        vals = {}
        for name, unit, v in zip(header, units, row):
            try:
                vals[name] = float(v.replace(",", "")) * _UNIT.get(unit, 1.0)
            except ValueError:
                pass
        out.append(vals)
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("csv")
    ap.add_argument("--kernel", required=True, choices=sorted(KERNEL_SOURCES))
    ap.add_argument("--workload", required=True)
    ap.add_argument("--units-per-launch", type=int, default=1, help="layer passes one captured launch processes")
    ap.add_argument("--note", default="")
    ap.add_argument("--per-workload", action="store_true",
                    help="write traffic_<kernel>_<workload>.txt (a second workload's record beside the kernel's first)")
    args = ap.parse_args(argv)
    launches = read_raw_csv(args.csv, args.kernel)
    if not launches:
        sys.exit(f"no launch of {args.kernel} in {args.csv}")
    rd = [l["dram__bytes_read.sum"] for l in launches]
    wr = [l["dram__bytes_write.sum"] for l in launches]
    per_unit = (sum(rd) + sum(wr)) / len(launches) / args.units_per_launch
    name = f"traffic_{args.kernel}_{args.workload}.txt" if args.per_workload else f"traffic_{args.kernel}.txt"
    path = os.path.join(ROOT, "profiles", name)
    with open(path, "w") as f:
        f.write("# DRAM traffic of one kernel from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),\n"
                "# written by python -m paper_2502_19078_b200.ncu_summary; bench.py reports it while the hash matches.\n")
        f.write(f"kernel: {args.kernel}\nworkload: {args.workload}\nnote: {args.note}\n")
        f.write(f"launches_captured: {len(launches)}\nunits_per_launch: {args.units_per_launch}\n")
        f.write(f"dram_bytes_read_per_unit: {sum(rd) / len(launches) / args.units_per_launch:.0f}\n")
        f.write(f"dram_bytes_write_per_unit: {sum(wr) / len(launches) / args.units_per_launch:.0f}\n")
        f.write(f"dram_bytes_per_unit: {per_unit:.0f}\n")
        f.write(f"sources: {' '.join(KERNEL_SOURCES[args.kernel])}\nsources_sha256: {sources_hash(args.kernel)}\n")
    print(path)


if __name__ == "__main__":
    main()
