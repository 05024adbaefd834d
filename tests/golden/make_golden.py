"""Writes tests/golden/oracle_cfg1.txt: oracle entropies and head outputs on the cfg1 workload.

Calls only the oracle (and the seeded input generator). The paper prints no numeric worked
example of an entropy value or a head output, so there are no paper-sourced fixtures; this
file is a regression guard on the oracle's own arithmetic. Values are stored as C99 hex floats.

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
import synth  # noqa: E402


def main():
    wl = synth.workload("cfg1")
    H = oracle.entropy(synth.features(wl))
    w = synth.head_weights(wl)
    toks = np.array([0, 1, 31, 63], np.int32)
    out = oracle.head_sample(w, synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K), toks)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_cfg1.txt")
    with open(path, "w") as f:
        f.write("# oracle values on workload cfg1 (written by make_golden.py; oracle-only)\n")
        f.write("# H <token> <entropy>   |   out <token> <channel> <x^K>\n")
        for i in range(0, wl.n, 8):
            f.write(f"H {i} {float(H[i]).hex()}\n")
        for t in toks:
            for c in range(0, wl.C, 5):
                f.write(f"out {int(t)} {c} {float(out[t, c]).hex()}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
