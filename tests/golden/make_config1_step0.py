"""Writes tests/golden/config1_step0.txt: per-subgraph loss, sum of probabilities, set size and
conflict counts of configuration 1 (G(1000, 0.01), 8 contiguous parts, 64-32-1) at its seeded
initial weights, computed by the float64 oracle only (Eqs. 3-5; decoding of Section 3.3).

The paper prints no worked numeric example of this path, so there is no value of the paper's to
store; this file is a drift guard: a later change to the oracle's arithmetic or to the input
generators shows up as a diff here and has to be justified.  Run from the repository root:

    python tests/golden/make_config1_step0.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import synth_inputs as si  # noqa: E402


def compute():
    w = si.make_workload(1)
    book = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    X = w.features_f32()[book["perm"]]
    W = [w.weights(l) for l in range(w.L)]
    r = oracle.train_step(book, w.dims, X, W, w.alpha, w.beta)
    d = oracle.decode(book, r["p"].astype(np.float32))
    psum = np.add.reduceat(r["p"], book["part_ptr"][:-1])
    return r["loss"], psum, d


def lines():
    loss, psum, d = compute()
    out = ["# subgraph  loss (Eq. 5, alpha=2, beta=1)  sum of p (Eq. 4)"]
    for s, (a, b) in enumerate(zip(loss, psum)):
        out.append("%d %.12e %.12e" % (s, a, b))
    out.append("# set size, intra conflicts, boundary conflicts (threshold 0.5 on float32 p)")
    out.append("%d %d %d" % (d["set_size"], d["intra_viol"], d["boundary_viol"]))
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_step0.txt")
    with open(path, "w") as f:
        f.write("\n".join(lines()) + "\n")
    print("wrote", path)
