"""Writes tests/golden/scan_tiny.txt: the oracle's outputs on a tiny seeded problem, as text.

The paper prints no worked numerical example of the scan, so there is no value of the paper's to store; this file is a
regression anchor of the ORACLE ONLY (it calls nothing but oracle/ and the seeded input generator), so that an
unintended change to the oracle's arithmetic shows up as a diff.  Run from the repository root:
    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ssm_oracle as O  # noqa: E402
from paper_2312_00752_b200 import synth  # noqa: E402  (input generator only: holds none of the method's arithmetic)


def tiny_problem():
    cfg = synth.ScanConfig("golden_tiny", 99, 1, 6, 2, 4, "f32", 1e-2, 1.0)
    return synth.make_inputs(cfg, seed=0)


def compute():
    p = tiny_problem()
    out = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"])
    g = O.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], p["dout"])
    zo = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"], zoh=True)
    return {"out": out, "out_zoh": zo, "dx": g["dx"], "ddelta": g["ddelta"], "dA": g["dA"], "dB": g["dB"],
            "dC": g["dC"], "dD": g["dD"], "dz": g["dz"]}


def main():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "scan_tiny.txt")
    with open(path, "w") as f:
        f.write("# oracle outputs for synth.ScanConfig('golden_tiny', 99, 1, 6, 2, 4, 'f32', 1e-2, 1.0), seed 0\n")
        f.write("# written by tests/golden/make_golden.py (calls only oracle/); one tensor per line: name shape values\n")
        for k, v in compute().items():
            v = np.asarray(v, dtype=np.float64)
            f.write(k + " " + "x".join(map(str, v.shape)) + " " + " ".join(repr(float(t)) for t in v.reshape(-1)) + "\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
