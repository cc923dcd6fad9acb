"""Writes tests/golden/oracle_regression.txt: a few outputs of the fp64 oracle on one small seeded case.

The file guards the ORACLE against accidental drift (a change of its arithmetic must be deliberate and
must regenerate this file); it is produced by the oracle alone -- nothing from the CUDA path enters it.
Run from the repository root:  python tests/golden/make_oracle_regression.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import flashbev_oracle  # noqa: E402
from paper_2607_10071_b200 import workloads as wl  # noqa: E402


def case():
    w = wl.Workload("golden", 900, 1, 6, 4, "f32", (6, 9), (48, 72), (7, 6, 5),
                    (-6.0, 6.0, -6.0, 6.0, -2.0, 2.5), 0, general_pose=True)
    return wl.make_inputs(w)


def rows():
    inp = case()
    w = inp.workload
    out = []
    for reduce in (0, 1, 2):
        r = flashbev_oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
        for (ix, iy, c) in ((0, 0, 0), (3, 2, 1), (6, 5, 3), (2, 4, 2), (5, 1, 0)):
            out.append((reduce, ix, iy, c, int(r.count[0, ix, iy]), float(r.out[0, ix, iy, c])))
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_regression.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_oracle_regression.py (oracle only): reduce ix iy c count value\n")
        for row in rows():
            f.write("%d %d %d %d %d %.17g\n" % row)
    print("wrote", path)
