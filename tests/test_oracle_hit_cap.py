"""Pins of the oracle's hit cap: compositing only the first m hits of a ray must equal compositing hit lists that were
cut to m hits by hand (a path that knows nothing of the cap), for the colour, T_final, the gradient and the
intermediate-buffer entries; hits behind the cap weigh nothing."""
import numpy as np
import pytest

import gart_scenes as gs
from oracle import gart_oracle as orc


def _truncate(ray_off, gid, m):
    cnt = np.diff(ray_off).astype(np.int64)
    keep = np.minimum(cnt, m)
    new_off = np.zeros(ray_off.size, dtype=np.uint64)
    new_off[1:] = np.cumsum(keep)
    idx = np.concatenate([np.arange(int(ray_off[r]), int(ray_off[r]) + int(keep[r])) for r in range(cnt.size)])
    return new_off, gid[idx], idx


@pytest.mark.parametrize("m", [1, 3, 8])
def test_cap_equals_truncated_lists(m):
    sc, cams = gs.config_tiny(sh_degree=2, seed=4)
    cam = cams[0]
    osc = orc.OracleScene.from_scene(sc)
    bg = (0.3, 0.2, 0.7)
    g = gs.upstream_gradient(cam, 1).astype(np.float64)
    full = orc.View(osc, cam, bg=bg)
    full.find_hits()
    ray_off, gid, _, _ = full.hits()
    assert np.diff(ray_off).max() > 8

    capped = orc.View(osc, cam, bg=bg, max_hits=m)
    capped.set_hits(ray_off, gid)
    c1, t1, n1 = capped.composite()
    g1, a1 = capped.backward(g, with_abs=True)
    e1, f1 = capped.lt_entries()

    cut = orc.View(osc, cam, bg=bg)
    off2, gid2, idx = _truncate(ray_off, gid, m)
    cut.set_hits(off2, gid2)
    c2, t2, n2 = cut.composite()
    g2, a2 = cut.backward(g, with_abs=True)
    e2, f2 = cut.lt_entries()

    assert np.array_equal(c1, c2) and np.array_equal(t1, t2)          # same arithmetic, hit for hit
    assert np.array_equal(n1.reshape(-1), np.diff(ray_off).astype(np.uint32))   # the lists still hold every hit
    assert np.all(np.abs(g1 - g2) <= 1e-12 * np.maximum(a1, a2))      # (threads add in varying order)
    assert np.allclose(a1, a2, rtol=1e-12, atol=0)
    # entries: those of the composited hits agree, the others are zero
    assert np.array_equal(e1[idx], e2) and np.array_equal(f1[idx], f2)
    dropped = np.ones(gid.size, bool)
    dropped[idx] = False
    assert dropped.any() and np.all(e1[dropped] == 0.0)
    # and the cap does change the view
    c0, t0, _ = full.composite()
    assert np.abs(c0 - c1).max() > 1e-3 and np.all(t1 >= t0)


def test_cap_larger_than_every_ray_changes_nothing():
    sc, cams = gs.config_tiny(seed=2)
    cam = cams[0]
    osc = orc.OracleScene.from_scene(sc)
    g = gs.upstream_gradient(cam, 0).astype(np.float64)
    a = orc.View(osc, cam)
    a.find_hits()
    lists = a.hits()[:2]
    b = orc.View(osc, cam, max_hits=10_000)
    b.set_hits(*lists)
    ca, ta, _ = a.composite()
    cb, tb, _ = b.composite()
    assert np.array_equal(ca, cb) and np.array_equal(ta, tb)
    ga, aa = a.backward(g, with_abs=True)
    gb = b.backward(g)
    assert np.all(np.abs(ga - gb) <= 1e-12 * aa)
