"""DRAM traffic per launch of the library's GEMM kernels, as measured by Nsight Compute.

bench.py reports, beside each roofline entry, the bytes one launch really moved to and from HBM
(dram__bytes_read.sum + dram__bytes_write.sum).  Those counters cannot be read while timing, so
they come from a separate capture of the same workload, kept in ncu_traffic.json next to this
file together with a digest of the kernel sources they were taken from.  `load()` hands the
numbers out only while the sources still have that digest: once a kernel changes, the traffic
figure is gone (None) until a new capture is recorded.

Recording (run the capture on a machine with a B200, then this tool on its CSV, with the sources unchanged in between):

    python bench.py --profile fused --config 2 --warmup 1 --steps 1          # plain run first, must exit 0
    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --clock-control none \\
        -k regex:gemm_kernel --csv --log-file traffic_fused.csv python bench.py --profile fused --config 2 --warmup 1 --steps 1
    python -m paper_2605_08632_b200.ncu_traffic record traffic_fused.csv --workload config2 --rows 16384 --path fused

Launches are matched to stages by the kernel's template arguments (operand majors and epilogue)
and taken from the LAST step in the capture, in launch order (row slab by row slab).
"""
from __future__ import annotations

import csv
import hashlib
import json
import os

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
STORE = os.path.join(PKG_DIR, "ncu_traffic.json")
SOURCES = ["csrc/cat_api.cu", "csrc/tc_gemm.cuh", "csrc/ptx.cuh", "csrc/rowops.cuh", "csrc/kd.cuh", "csrc/simt.cuh"]

# kernel-name fragment -> stage name
STAGE_OF = {
    "gemm_kernel<0, 0, EpiFwdT<2>": "logits",
    "gemm_kernel<0, 1, EpiOut": "dH",
    "gemm_kernel<1, 1, EpiOut": "dW",
    "gemm_kernel<0, 0, EpiFwdT<0>": "fwd_two_call",
    "gemm_kernel<0, 0, EpiDz": "dz_two_call",
}


def source_digest() -> str:
    h = hashlib.sha256()
    for rel in SOURCES:
        with open(os.path.join(PKG_DIR, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def parse(csv_path: str) -> list:
    """[(stage, {metric: value})] per captured launch, in launch order."""
    launches, hdr = {}, None
    with open(csv_path, newline="") as f:
        for r in csv.reader(f):
            if r and r[0] == "ID":
                hdr = r
                continue
            if hdr and len(r) == len(hdr):
                d = dict(zip(hdr, r))
                name = d["Kernel Name"].replace("cat::", "").replace("tc::", "")      # ncu may or may not print namespaces
                stage = next((s for frag, s in STAGE_OF.items() if frag in name), None)
                if stage is None:
                    continue
                ent = launches.setdefault(int(d["ID"]), (stage, {}))
                ent[1][d["Metric Name"]] = float(d["Metric Value"].replace(",", ""))
    return [launches[k] for k in sorted(launches)]


def record(csv_path: str, workload: str, rows: int, path: str) -> dict:
    per_stage = {}
    for stage, m in parse(csv_path):
        if "dram__bytes_read.sum" in m and "dram__bytes_write.sum" in m:
            per_stage.setdefault(stage, []).append(dict(read=m["dram__bytes_read.sum"], write=m["dram__bytes_write.sum"],
                                                        ns=m.get("gpu__time_duration.sum")))
    store = json.load(open(STORE)) if os.path.exists(STORE) else {}
    ent = store.setdefault(f"{workload}:{rows}:{path}", {})
    ent["source_digest"] = source_digest()
    ent["csv"] = os.path.basename(csv_path)
    ent["stages"] = per_stage
    with open(STORE, "w") as f:
        json.dump(store, f, indent=1, sort_keys=True)
    return ent


def load(workload: str, rows: int, path: str):
    """{stage: [ {read, write, ns} per launch of the last captured step ]} or None when there is no
    capture for this workload or the kernel sources changed since it was taken."""
    if not os.path.exists(STORE):
        return None
    ent = json.load(open(STORE)).get(f"{workload}:{rows}:{path}")
    if not ent or ent.get("source_digest") != source_digest():
        return None
    return ent["stages"]


def bytes_of(stages, stage: str, launch: int = 0, n_launches_per_step: int | None = None):
    """read + write bytes of launch `launch` (index within a step) of `stage`, or None."""
    if not stages or stage not in stages:
        return None
    ls = stages[stage]
    if n_launches_per_step:
        ls = ls[-n_launches_per_step:]            # the last captured step
    if launch >= len(ls):
        return None
    return int(ls[launch]["read"] + ls[launch]["write"])


if __name__ == "__main__":
    import argparse
    ap = argparse.ArgumentParser()
    ap.add_argument("cmd", choices=["record", "show"])
    ap.add_argument("csv", nargs="?")
    ap.add_argument("--workload", default="config2")
    ap.add_argument("--rows", type=int, default=16384)
    ap.add_argument("--path", default="fused", choices=["fused", "two-call"])
    a = ap.parse_args()
    if a.cmd == "record":
        e = record(a.csv, a.workload, a.rows, a.path)
        for st, ls in e["stages"].items():
            for i, l in enumerate(ls):
                print(f"{st}[{i}]: read {l['read'] / 1e9:.3f} GB  write {l['write'] / 1e9:.3f} GB  {(l['ns'] or 0) / 1e6:.3f} ms")
    else:
        print(json.dumps(load(a.workload, a.rows, a.path), indent=1))
