"""Writes tests/golden/cfg1_oracle_values.txt: values of the CPU oracle on the smallest configured workload (cfg1),
sampled at fixed positions, so that a later change to the oracle's arithmetic shows up as a difference against a stored
file and has to be justified.  The paper prints no worked numeric example of the layer (its Methods define
y = x W + s_t (x A_t) B_t for every token of tenant t and train the adapters by back-propagation), so there is no printed
value to store; these are the oracle's own, written by this script, which calls only the seeded input generators and
oracle/.  Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2605_08527_b200 import workloads as wl  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_oracle_values.txt")


def sample_positions(shape, n, salt):
    """n fixed positions of an array of this shape (a plain multiplicative walk: no library generator involved)."""
    size = int(np.prod(shape))
    idx = [(salt * 7919 + k * 104729) % size for k in range(n)]
    return [tuple(int(v) for v in np.unravel_index(i, shape)) for i in idx]


def oracle_values():
    """name -> (array, sampled positions) for every output of the oracle on cfg1, in float64."""
    w = wl.make_workload(1)
    p = w.projections[0]
    ts = w.tok_slot()
    r, s, A, B = oracle.adapters_of(p, np.float64)
    y, h = oracle.forward(p.x, p.W, r, s, A, B, ts, dtype=np.float64)
    Tb = p.dy.shape[0]
    dx, g = oracle.backward_dx(p.dy, p.W, r, s, A, B, ts[:Tb], dtype=np.float64)
    dA, dB = oracle.backward_dAdB(p.x[:Tb], p.dy, r, s, A, B, ts[:Tb], dtype=np.float64)
    out = {"y": y, "h": h, "dx": dx, "g": g}
    for t in range(len(p.adapters)):
        if r[t] > 0:
            out[f"dA[{t}]"] = dA[t]
            out[f"dB[{t}]"] = dB[t]
    return {k: (np.asarray(v, np.float64), sample_positions(np.shape(v), 6, 1 + i)) for i, (k, v) in enumerate(out.items())}


def lines():
    yield "# oracle values on cfg1 (float64), written by tests/golden/make_golden.py; name, index, value; 'sum' = sum of all entries"
    for name, (arr, pos) in oracle_values().items():
        yield f"{name} shape {' '.join(str(d) for d in arr.shape)}"
        yield f"{name} sum {float(arr.sum()):.17g}"
        for ix in pos:
            yield f"{name} at {' '.join(str(i) for i in ix)} {float(arr[ix]):.17g}"


if __name__ == "__main__":
    with open(OUT, "w") as f:
        f.write("\n".join(lines()) + "\n")
    print("wrote", OUT)
