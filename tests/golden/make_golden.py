"""Writes tests/golden/qdelta_tiny.txt: forward and reverse-pass results of the fp64 oracle on one tiny,
seeded problem.  Calls nothing but `oracle/` and the seeded input generator; run from the repository root:

    python tests/golden/make_golden.py

The file guards the oracle against unintended changes (the pins in tests/test_oracle_*.py are what ties it
to the paper).  The paper itself prints no numerical example of the update rule, so no value here is the
paper's.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import recurrence  # noqa: E402
from paper_2606_08804_b200 import inputs as gen  # noqa: E402

CFG = gen.Config("golden_tiny", 1, 6, 2, 3, 2, 64, "f32", True, True, seed=1234)


def compute():
    d = gen.make_chunk_inputs(CFG)
    o, hT = recurrence.forward(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"])
    g = recurrence.backward(d["q"], d["k"], d["v"], d["beta"], d["alpha"], d["lam"], d["h0"], d["dO"], d["dhT"])
    out = {"o": o, "hT": hT}
    for n in ("dq", "dk", "dv", "dbeta", "dalpha", "dlam", "dh0"):
        out[n] = g[n]
    return out


def main():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "qdelta_tiny.txt")
    with open(path, "w") as f:
        f.write("# oracle results for Config%r; written by tests/golden/make_golden.py\n" % (tuple(CFG.__dict__.values()),))
        for n, v in compute().items():
            v = np.asarray(v, np.float64)
            f.write("%s %s\n" % (n, " ".join(str(x) for x in v.shape)))
            f.write(" ".join("%.17g" % x for x in v.ravel()) + "\n")
    print(path)


if __name__ == "__main__":
    main()
