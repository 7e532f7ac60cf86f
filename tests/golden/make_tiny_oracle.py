"""Writes tests/golden/tiny_oracle.txt: digests of the oracle's view of the Tiny configuration (64 x 64 pixels, 256 Gaussians,
SH degree 0, seed 0).  Calls only the oracle and the seeded scene generator.  The file is a regression pin: it holds no
independent truth (the oracle's pins are in tests/test_oracle_*.py), it makes a later change of the oracle's arithmetic
visible, and the GPU path is compared with the same stored numbers.

    python tests/golden/make_tiny_oracle.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
import gart_scenes as gs  # noqa: E402
from oracle import gart_oracle as orc  # noqa: E402


def digests():
    scene, cams = gs.config_tiny()
    cam = cams[0]
    g = gs.upstream_gradient(cam, 0).astype(np.float64)
    out = orc.render(orc.OracleScene.from_scene(scene), cam, dL_dC=g, alpha_min=float(np.float32(1.0 / 255.0)), near=float(np.float32(0.01)))
    grad = out["grad"]
    rows = [("hits", float(out["hit_count"].sum())), ("max_hits_per_ray", float(out["hit_count"].max()))]
    for c in range(3):
        rows.append(("sum_color_%d" % c, float(out["color"][..., c].sum())))
    rows.append(("sum_t_final", float(out["t_final"].sum())))
    names = ["mean_x", "mean_y", "mean_z", "scale_x", "scale_y", "scale_z", "quat_w", "quat_x", "quat_y", "quat_z", "opacity", "dc_r", "dc_g", "dc_b"]
    for j, nme in enumerate(names):
        rows.append(("sum_abs_grad_" + nme, float(np.abs(grad[:, j]).sum())))
    for y, x in ((10, 12), (31, 33), (50, 7)):
        for c in range(3):
            rows.append(("color_%d_%d_%d" % (y, x, c), float(out["color"][y, x, c])))
    return rows


if __name__ == "__main__":
    with open(os.path.join(HERE, "tiny_oracle.txt"), "w") as f:
        f.write("# written by tests/golden/make_tiny_oracle.py from the oracle alone (Tiny: 64 x 64, 256 Gaussians, SH degree 0, seed 0)\n")
        for k, v in digests():
            f.write("%s %.17g\n" % (k, v))
    print("written")
