"""Stored values: what the paper prints for the hot path (tests/golden/paper_constants.txt, each line cited) against the
library's constants and defaults, and the oracle-written digests of the Tiny configuration (tests/golden/tiny_oracle.txt,
written by tests/golden/make_tiny_oracle.py from the oracle alone) against the oracle as it stands and against the GPU path."""
import importlib.util
import os

import numpy as np
import pytest

import gart_scenes as gs
import paper_2608_17298_b200.gart as G

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _read(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def test_paper_constants_are_the_librarys():
    c = _read("paper_constants.txt")
    cfg = G.Config()
    assert np.float32(cfg.alpha_min) == np.float32(1.0 / c["alpha_min_denominator"])
    assert cfg.tile_size == c["tile_edge_pixels"] and cfg.kernel_degree == c["kernel_degree"]
    K = (3 + 1) ** 2
    assert 3 + 3 + 4 + 1 + 3 * K == c["gradient_words_sh3"] and 3 * K == c["sh_gradient_words_sh3"]
    assert G.GRAD_WORDS >= c["gradient_words_sh3"] and G.GRAD_WORDS % 4 == 0        # a record holds the 59 words, padded to whole 16-byte pieces
    assert cfg.lt_format == 0 and 4 * 4 == c["lt_entry_bytes"]                       # format 0: four floats per hit


def test_oracle_reproduces_its_stored_tiny_digests():
    spec = importlib.util.spec_from_file_location("make_tiny_oracle", os.path.join(GOLDEN, "make_tiny_oracle.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = _read("tiny_oracle.txt")
    now = dict(mod.digests())
    assert set(now) == set(stored)
    for k, v in stored.items():
        assert abs(now[k] - v) <= 1e-11 * max(abs(v), 1.0), (k, now[k], v)     # (threads sum in any order)


@pytest.mark.gpu
def test_gpu_path_meets_the_stored_tiny_digests():
    import parity as P
    stored = _read("tiny_oracle.txt")
    scene, cams = gs.config_tiny()
    cam = cams[0]
    gpu = P.run_gpu(scene, cam, G.Config(tile_size=16), gs.upstream_gradient(cam, 0))
    assert gpu["counts"][G.CNT_HITS] == stored["hits"] and gpu["hit_count"].max() == stored["max_hits_per_ray"]
    col = gpu["color"].astype(np.float64)
    for c in range(3):
        assert abs(col[..., c].sum() - stored["sum_color_%d" % c]) <= 1e-4 * stored["sum_color_%d" % c]
    assert abs(gpu["t_final"].astype(np.float64).sum() - stored["sum_t_final"]) <= 1e-4 * stored["sum_t_final"]
    for (y, x) in ((10, 12), (31, 33), (50, 7)):
        for c in range(3):
            v = stored["color_%d_%d_%d" % (y, x, c)]
            assert abs(col[y, x, c] - v) <= 1e-4 * abs(v) + 1e-7
    names = ["mean_x", "mean_y", "mean_z", "scale_x", "scale_y", "scale_z", "quat_w", "quat_x", "quat_y", "quat_z", "opacity", "dc_r", "dc_g", "dc_b"]
    for variant in ("grad", "grad_tile", "grad_atomic"):
        gr = np.abs(gpu[variant].astype(np.float64))
        for j, nme in enumerate(names):
            v = stored["sum_abs_grad_" + nme]
            assert abs(gr[:, j].sum() - v) <= 1e-3 * v, (variant, nme)
