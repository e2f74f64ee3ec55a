"""Record the DRAM traffic of one benchmark step from an ncu launch list.

    python -m paper_1804_10727_b200.record_traffic WORKLOAD N_STREAMS ROWS launches.csv

``launches.csv`` is the ``--csv`` log of an ``ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum``
capture of exactly one step's kernels (ROWS segments per stream).  The sum of both counters over all captured
launches, divided by ROWS, is stored in ``dram_traffic.json`` beside this file together with a fingerprint of
the CUDA sources, so that ``bench.py`` reports the figure only for the kernels it was measured on.
"""
import csv
import io
import json
import os
import sys


def main():
    name, n_streams, rows, path = sys.argv[1], int(sys.argv[2]), int(sys.argv[3]), sys.argv[4]
    txt = open(path).read()
    table = list(csv.DictReader(io.StringIO(txt[txt.index('"ID"'):])))
    total, launches = 0.0, set()
    for r in table:
        if r["Metric Name"] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            total += float(r["Metric Value"].replace(",", ""))
            launches.add(r["ID"])
    here = os.path.dirname(os.path.abspath(__file__))
    sys.path.insert(0, os.path.dirname(here))
    from bench import kernel_source_hash
    out = os.path.join(here, "dram_traffic.json")
    rec = json.load(open(out)) if os.path.exists(out) else {}
    rec[name] = {"kernel_source_hash": kernel_source_hash(), "n_streams": n_streams, "bytes_per_row": total / rows,
                 "note": f"dram__bytes_read.sum + dram__bytes_write.sum over the {len(launches)} launches of one {rows}-row step "
                         "(ncu, cold caches, launches serialised)"}
    json.dump(rec, open(out, "w"), indent=1)
    print(out, rec[name])


if __name__ == "__main__":
    main()
