"""Writes tests/golden/oracle_regression_c0.txt: a few dozen values of the oracle's own output
on the smallest workload (C0, seed 0) and on a small gate problem.

The paper prints no worked example for this path, so these are not the paper's numbers: they
freeze the oracle as it stood when its pins (tests/test_oracle_*_pins.py) were last checked, so
that an unintended edit of its arithmetic shows up as a diff here.  The script calls only
oracle/ and the seeded input generator; run it again (and say why in the commit) whenever the
oracle's arithmetic changes on purpose.

    python tests/golden/make_oracle_regression.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ssm_oracle as O  # noqa: E402
from paper_2502_20168_b200 import inputs as I  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_regression_c0.txt")


def values():
    d = I.draw_layer(I.C0)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    y, xT, _ = O.ssm_layer_fwd(*args, d["u"], d["done"], None)
    g = O.ssm_layer_bwd(*args, d["u"], d["done"], None, d["gy"])
    w = I.Workload("gate", B=2, T=5, H=16, P=8, io_dtype="f32", seed=11)
    q = I.draw_glu(w)
    out = O.half_glu_fwd(q["W"], q["v"])
    gv, dW = O.half_glu_bwd(q["W"], q["v"], q["gout"])
    rows = []

    def add(name, a, idx):
        v = np.asarray(a)[idx]
        if np.iscomplexobj(v):
            rows.append((f"{name}{list(idx)}.re", float(v.real)))
            rows.append((f"{name}{list(idx)}.im", float(v.imag)))
        else:
            rows.append((f"{name}{list(idx)}", float(v)))

    for idx in [(0, 0, 0), (0, 31, 7), (0, 63, 31)]:
        add("y", y, idx)
        add("du", g["du"], idx)
    for idx in [(0, 0), (0, 15)]:
        add("xT", xT, idx)
    for p in (0, 7, 15):
        add("dLambda", g["dLambda"], (p,))
        add("dDelta", g["dDelta"], (p,))
    for idx in [(0, 0), (15, 31)]:
        add("dB", g["dB"], idx)
        add("dC", g["dC"], idx[::-1])
    for h in (0, 31):
        add("dD", g["dD"], (h,))
    for idx in [(0, 0, 0), (1, 4, 15)]:
        add("glu_out", out, idx)
        add("glu_gv", gv, idx)
    for idx in [(0, 0), (15, 3)]:
        add("glu_dW", dW, idx)
    return rows


if __name__ == "__main__":
    with open(OUT, "w") as f:
        f.write("# oracle outputs, float64, written by tests/golden/make_oracle_regression.py (not values from the paper)\n")
        for name, v in values():
            f.write(f"{name} {v!r}\n")
    print(OUT)
