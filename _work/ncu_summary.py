"""Turn ncu launch-list CSVs into the text summary and the DRAM-traffic table kept under profiles/.

    python -m paper_2406_17611_b200.ncu_summary TIMES.csv DRAM.csv [--json OUT.json]

TIMES.csv: ncu --metrics gpu__time_duration.sum --csv --log-file TIMES.csv <cmd>
DRAM.csv : ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --csv --log-file DRAM.csv <cmd>
Both over the same launches of one epoch.  Kernels are mapped to the benchmark's stage names so that
bench.py can quote the measured DRAM traffic of a stage next to its algorithmic bytes.
"""
from __future__ import annotations

import collections
import csv
import hashlib
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
UNITS = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "ns": 1e-6, "us": 1e-3, "ms": 1.0, "s": 1e3}


def source_digest() -> str:
    """SHA-1 over the CUDA sources: a traffic table is only quoted for the kernels it was taken from."""
    h = hashlib.sha1()
    csrc = os.path.join(HERE, "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh", ".h", ".cpp")):
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()


def _load(path):
    rows = list(csv.reader(open(path)))
    i = [k for k, r in enumerate(rows) if r and r[0] == "ID"][0]
    return [dict(zip(rows[i], r)) for r in rows[i + 1:]]


def _short(name):
    return name.split("(")[0].replace("void ", "").replace("<unnamed>::", "")


def stage_of(kernels):
    """Stage of every launch of an epoch, from the order the layer entry points launch their kernels."""
    stages, seen_fwd_gemm, masked_colsum = [], 0, False
    n_layers = sum(1 for k in kernels if k.startswith("rows_kernel")) // 2
    for k in kernels:
        if k.startswith(("gather_copy", "compress_rows")):
            st = "compress"
        elif k.startswith(("decompress_slots", "decompress_brows", "expand_slots")):
            st = "decompress"
        elif k.startswith(("add_dense_rows", "scatter_add_rows")):
            st = "scatter_add"
        elif k.startswith("colsum"):
            # the masked form is the ReLU mask of the backward pass with the bias gradient fused in
            masked_colsum = k.replace(" ", "").endswith((",1>", ",true>"))
            st = "aux" if masked_colsum else "gemm_dw"
        elif k.startswith("reduce_partials"):
            st = "aux" if masked_colsum else "gemm_dw"
            masked_colsum = False
        elif k.startswith(("dw_kernel", "dw_reduce")):
            st = "gemm_dw"
        elif k.startswith(("wire_positions", "select_slots", "slot_kept_product")):
            st = "compress_bwd"
        elif k.startswith("relu_mask"):
            st = "aux"
        elif k.startswith("spmm"):
            st = "spmm" if seen_fwd_gemm < n_layers else "spmm_t"
        elif k.startswith(("rows_kernel", "pack_weights")):
            if k.startswith("rows_kernel"):
                seen_fwd_gemm += 1
            st = "gemm_fwd" if seen_fwd_gemm <= n_layers and not (k.startswith("pack") and seen_fwd_gemm == n_layers) \
                else "gemm_dx"
        else:
            st = "other"
        stages.append(st)
    return stages


def summarize(times_csv, dram_csv):
    t, d = _load(times_csv), _load(dram_csv)
    launches = collections.OrderedDict()
    for r in t:
        launches[r["ID"]] = dict(kernel=_short(r["Kernel Name"]), grid=r.get("Grid Size", ""),
                                 ms=float(r["Metric Value"].replace(",", "")) * UNITS[r["Metric Unit"]], rd=0.0, wr=0.0)
    for r in d:
        v = float(r["Metric Value"].replace(",", "")) * UNITS[r["Metric Unit"]]
        launches[r["ID"]]["rd" if "read" in r["Metric Name"] else "wr"] += v
    ids = sorted(launches, key=int)
    for i, st in zip(ids, stage_of([launches[i]["kernel"] for i in ids])):
        launches[i]["stage"] = st
    return [launches[i] for i in ids]


def render(rows):
    out = ["# per launch of one epoch: kernel, stage, grid, ms under ncu, DRAM read GB, DRAM write GB"]
    tot = sum(r["ms"] for r in rows)
    for i, r in enumerate(rows):
        out.append("%3d %-44s %-12s %-16s %8.3f %8.3f %8.3f" % (i, r["kernel"][:44], r["stage"], r["grid"], r["ms"],
                                                                 r["rd"] / 1e9, r["wr"] / 1e9))
    for key, title in (("kernel", "per kernel"), ("stage", "per stage")):
        agg = collections.OrderedDict()
        for r in rows:
            a = agg.setdefault(r[key], [0, 0.0, 0.0, 0.0])
            a[0] += 1
            a[1] += r["ms"]
            a[2] += r["rd"]
            a[3] += r["wr"]
        out.append("\n# %s: launches, total ms, share, DRAM read GB, write GB, DRAM GB/s (bytes / ncu time)" % title)
        for n, (c, ms, rd, wr) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
            out.append("%-44s %3d %8.3f %5.1f%% %8.2f %8.2f %8.0f" % (n[:44], c, ms, 100 * ms / tot, rd / 1e9, wr / 1e9,
                                                                     (rd + wr) / ms / 1e6))
    out.append("total ms %.3f launches %d" % (tot, len(rows)))
    return "\n".join(out)


def main(argv):
    rows = summarize(argv[0], argv[1])
    print(render(rows))
    if "--json" in argv:
        per_stage = collections.OrderedDict()
        for r in rows:
            per_stage[r["stage"]] = per_stage.get(r["stage"], 0.0) + r["rd"] + r["wr"]
        json.dump({"source_sha1": source_digest(), "dram_bytes_per_epoch": per_stage},
                  open(argv[argv.index("--json") + 1], "w"), indent=1)


if __name__ == "__main__":
    main(sys.argv[1:])
