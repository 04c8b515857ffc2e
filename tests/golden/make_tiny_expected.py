"""Writes tests/golden/tiny_adam_expected.txt: the oracle's result for the "tiny" workload
(6 tensors, R=4, Adam, step 10, seed 0, inputs drawn on the CPU).  Calls only the oracle and
the seeded input generators; run it again only when the oracle's arithmetic changes for a
reason the paper supports.

    python tests/golden/make_tiny_expected.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ws_oracle as O                      # noqa: E402
from paper_2004_13336_b200 import workloads as W       # noqa: E402


def main():
    wl = W.tiny()
    w, m, v = [[x.numpy() for x in lst] for lst in W.make_state(wl, "cpu")]
    g = [[x.numpy() for x in gk] for gk in W.make_grads(wl, "cpu")]
    O.update_unsharded(O.make_hyper(wl.opt, wl.hyper), g, w, m, v)
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_adam_expected.txt")
    with open(out, "w") as f:
        f.write("# Oracle (unsharded definition, Section 2.2: all replicas sum gradients and apply the same\n")
        f.write("# update) on the tiny workload: per tensor and per output (w', m', v') the element count, the\n")
        f.write("# float64 sum, the float64 sum of squares, and elements 0, n//3, 2n//3, n-1 as float32 hex.\n")
        for name, lst in (("w", w), ("m", m), ("v", v)):
            for t, x in enumerate(lst):
                n = x.size
                picks = [0, n // 3, 2 * n // 3, n - 1]
                hexes = " ".join(float(x[i]).hex() for i in picks)
                f.write(f"{name} {t} {n} {float(x.astype(np.float64).sum())!r} "
                        f"{float((x.astype(np.float64) ** 2).sum())!r} {hexes}\n")
    print("wrote", out)


if __name__ == "__main__":
    main()
