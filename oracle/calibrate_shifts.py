"""Calibrate the requantisation shifts of the int8 workloads on the CPU oracle.

For each conv layer in turn: the smallest shift such that the 99.9th percentile
of the rounded, shifted ReLU output stays at or below 127.  Prints the tuples
that are frozen in paper_1804_10727_b200/workloads.py (_SHIFTS).

Run:  python -m oracle.calibrate_shifts
"""
from dataclasses import replace

import numpy as np

from oracle import oracle
from paper_1804_10727_b200 import workloads


def calibrate(name: str, n_streams: int):
    w = workloads.get(name, n_streams=n_streams)
    x = workloads.make_input(w).astype(np.int32)
    ws, _ = workloads.make_params(w)
    a = x
    shifts = []
    for l, wt in zip(w.layers, ws):
        if l.kind == "pool":
            a = oracle.pool_layer("i8", a)
            continue
        c = oracle.conv_layer("i8", l, a, wt, None)
        shift = 0
        while True:
            q = (c.astype(np.int64) + ((1 << (shift - 1)) if shift > 0 else 0)) >> shift
            if np.percentile(q, 99.9) <= 127:
                break
            shift += 1
        shifts.append(shift)
        a = oracle.requant(c, shift, l.relu)
        nz = float((a != 0).mean())
        print(f"  {name}: conv {l.cin}->{l.cout} shift {shift}  max c {int(c.max())}  non-zero fraction {nz:.3f}")
    return tuple(shifts)


if __name__ == "__main__":
    print("mnist2d", calibrate("mnist2d", 256))
    print("events2d", calibrate("events2d", 8))
