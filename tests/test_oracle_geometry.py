"""Pins for the oracle's geometry: SH table, bounds (Eq. 11-14), tile map, t* (Eq. 4-5).

Every expected value here comes from mathematics or from a library routine that the
oracle does not call: scipy's complex spherical harmonics, scipy's quaternion
rotation, dense projection of ellipsoid surface points, the tangent-line bound of
a sphere, a golden-section search, and a numpy overlap test.
"""
import math

import numpy as np
import pytest
from scipy.optimize import minimize_scalar
from scipy.spatial.transform import Rotation

import gart_scenes as gs
from oracle import gart_oracle as orc

AMIN = 1.0 / 255.0


def _fib_sphere(n):
    i = np.arange(n) + 0.5
    phi = np.arccos(1 - 2 * i / n)
    th = math.pi * (1 + 5 ** 0.5) * i
    return np.stack([np.cos(th) * np.sin(phi), np.sin(th) * np.sin(phi), np.cos(phi)], axis=1)


def _rot(q_wxyz):
    w, x, y, z = q_wxyz
    return Rotation.from_quat([x, y, z, w]).as_matrix()


# ------------------------------------------------------------------ SH table
def test_sh_matches_complex_harmonics():
    """Y_k = sqrt(2) Re/Im of the complex harmonics (Condon-Shortley phase kept): pins signs and constants."""
    from scipy.special import sph_harm_y
    rng = np.random.default_rng(1)
    for _ in range(50):
        d = rng.standard_normal(3)
        d /= np.linalg.norm(d)
        theta, phi = math.acos(d[2]), math.atan2(d[1], d[0])
        Y = orc.sh_basis(d)
        for l in range(4):
            for m in range(-l, l + 1):
                ylm = sph_harm_y(l, abs(m), theta, phi)
                ref = ylm.real if m == 0 else math.sqrt(2) * (ylm.real if m > 0 else ylm.imag)
                assert Y[l * (l + 1) + m] == pytest.approx(ref, abs=1e-13)


def test_sh_unsoeld_and_orthonormal():
    pts = _fib_sphere(200)
    Y = np.stack([orc.sh_basis(p) for p in pts])
    for l in range(4):
        s = (Y[:, l * l:(l + 1) * (l + 1)] ** 2).sum(axis=1)
        assert np.allclose(s, (2 * l + 1) / (4 * math.pi), atol=1e-14)
    # Gauss-Legendre in cos(theta) x uniform in phi integrates degree-6 polynomials exactly
    xs, ws = np.polynomial.legendre.leggauss(8)
    G = np.zeros((16, 16))
    nphi = 16
    for ct, w in zip(xs, ws):
        st = math.sqrt(1 - ct * ct)
        for j in range(nphi):
            ph = 2 * math.pi * j / nphi
            y = orc.sh_basis(np.array([st * math.cos(ph), st * math.sin(ph), ct]))
            G += w * (2 * math.pi / nphi) * np.outer(y, y)
    assert np.allclose(G, np.eye(16), atol=1e-12)


# ------------------------------------------------------------------ rays
def test_ray_convention():
    cam = gs.pinhole(64, 48, 50.0, gs.look_at((1.0, -2.0, 3.0), (0.2, 0.1, -0.3)))
    o, d = orc.ray(cam, 10, 7)
    R, t = cam.w2c[:, :3], cam.w2c[:, 3]
    assert np.allclose(R @ o + t, 0, atol=1e-14)            # the origin maps to the camera centre
    dc = R @ d
    assert dc[2] > 0 and abs(np.linalg.norm(d) - 1) < 1e-15
    assert cam.fx * dc[0] / dc[2] + cam.cx == pytest.approx(10.5, abs=1e-12)
    assert cam.fy * dc[1] / dc[2] + cam.cy == pytest.approx(7.5, abs=1e-12)


# ------------------------------------------------------------------ bounds
def _one(mean, scale, quat, opacity, deg=0):
    K = (deg + 1) ** 2
    n = len(opacity)
    return orc.OracleScene(np.array(mean, float).reshape(n, 3), np.array(scale, float).reshape(n, 3),
                           np.array(quat, float).reshape(n, 4), np.array(opacity, float), np.full((n, K, 3), 0.3), deg)


def test_bounds_sphere_tangent_lines():
    """Isotropic Gaussian = sphere of radius alpha_c * s: its exact screen extent is given by tangent lines."""
    rng = np.random.default_rng(2)
    cam = gs.pinhole(400, 300, 70.0)
    n = 300
    mean = np.stack([rng.uniform(-2, 2, n), rng.uniform(-1.5, 1.5, n), rng.uniform(2, 6, n)], 1)
    s = rng.uniform(0.01, 0.3, n)
    op = rng.uniform(0.05, 0.99, n)
    sc = _one(mean, np.repeat(s[:, None], 3, 1), _unit_q(rng, n), op)
    rect, cls, margin = orc.bounds(sc, cam)
    checked = 0
    for i in range(n):
        r = math.sqrt(2 * math.log(op[i] / AMIN)) * s[i]
        X, Y, Z = mean[i]
        assert cls[i] == 1
        exp = []
        for (a, f, c, lim) in ((X, cam.fx, cam.cx, cam.width), (Y, cam.fy, cam.cy, cam.height)):
            th, ph = math.atan2(a, Z), math.asin(r / math.hypot(a, Z))
            lo, hi = f * math.tan(th - ph) + c, f * math.tan(th + ph) + c
            exp.append((max(0, math.ceil(lo - 0.5)), min(lim - 1, math.floor(hi - 0.5))))
        if margin[i] < 1e-7:
            continue
        (x0, x1), (y0, y1) = exp
        want = [x0, y0, x1, y1] if (x1 >= x0 and y1 >= y0) else [0, 0, -1, -1]
        assert list(rect[i]) == want, (i, rect[i], want)
        checked += 1
    assert checked > 250


def _unit_q(rng, n):
    q = rng.standard_normal((n, 4))
    return q / np.linalg.norm(q, axis=1, keepdims=True)


def test_bounds_enclose_and_are_tight_on_projected_ellipsoid():
    """Dense surface samples of the alpha_c-ellipsoid, projected: the rectangle is their pixel-centre hull."""
    rng = np.random.default_rng(3)
    cam = gs.pinhole(640, 480, 60.0, gs.look_at((0.3, -0.2, -4.0), (0.0, 0.1, 0.0)))
    n = 60
    mean = rng.uniform(-1.0, 1.0, (n, 3))
    scale = np.exp(rng.uniform(math.log(0.02), math.log(0.4), (n, 3)))
    quat = _unit_q(rng, n)
    op = rng.uniform(0.05, 0.99, n)
    sc = _one(mean, scale, quat, op)
    rect, cls, margin = orc.bounds(sc, cam)
    u = _fib_sphere(200_000)
    Rc, tc = cam.w2c[:, :3], cam.w2c[:, 3]
    exact = 0
    for i in range(n):
        ac = math.sqrt(2 * math.log(op[i] / AMIN))
        pts = mean[i] + (u * (scale[i] * ac)) @ _rot(quat[i]).T
        pc = pts @ Rc.T + tc
        assert cls[i] == 1 and pc[:, 2].min() > 0.01
        px = cam.fx * pc[:, 0] / pc[:, 2] + cam.cx
        py = cam.fy * pc[:, 1] / pc[:, 2] + cam.cy
        sx0, sx1 = max(0, math.ceil(px.min() - 0.5)), min(cam.width - 1, math.floor(px.max() - 0.5))
        sy0, sy1 = max(0, math.ceil(py.min() - 0.5)), min(cam.height - 1, math.floor(py.max() - 0.5))
        x0, y0, x1, y1 = rect[i]
        if sx1 < sx0 or sy1 < sy0:
            continue
        # conservative: contains every sampled surface point's pixel; tight: at most the one pixel
        # column/row that the finite sampling can miss
        assert x0 <= sx0 and y0 <= sy0 and x1 >= sx1 and y1 >= sy1
        assert sx0 - x0 <= 1 and sy0 - y0 <= 1 and x1 - sx1 <= 1 and y1 - sy1 <= 1
        exact += [x0, y0, x1, y1] == [sx0, sy0, sx1, sy1]
    assert exact >= 0.9 * n


def test_bounds_classes():
    cam = gs.pinhole(64, 64, 50.0)
    q = [1, 0, 0, 0]
    sc = _one([[0, 0, 3], [0, 0, 3], [0, 0, -3], [0, 0, 0.2], [30, 0, 0.2], [40, 0, 3]],
              [[0.1] * 3, [0.1] * 3, [0.1] * 3, [0.5] * 3, [0.5] * 3, [0.1] * 3], [q] * 6,
              [0.5, AMIN, 0.5, 0.9, 0.9, 0.9])
    rect, cls, _ = orc.bounds(sc, cam)
    assert list(cls) == [1, 0, 0, 2, 2, 1]
    assert list(rect[3]) == [0, 0, 63, 63]       # straddles the camera plane, inside the frustum
    assert list(rect[4]) == [0, 0, -1, -1]       # straddles, but its sphere is outside a side plane
    assert list(rect[5]) == [0, 0, -1, -1]       # in front, off screen
    assert list(rect[1]) == [0, 0, -1, -1] and list(rect[2]) == [0, 0, -1, -1]


def test_hits_lie_inside_rectangles():
    """Conservativeness: every brute-force hit pixel is inside its Gaussian's rectangle."""
    for sc, cams in (gs.config_tiny(), gs.config_cluster(n=300, width=64, height=64)):
        osc = orc.OracleScene.from_scene(sc)
        rect, cls, _ = orc.bounds(osc, cams[0])
        v = orc.View(osc, cams[0])
        assert v.find_hits(orc.BRUTE) > 1000
        ray_off, gid, _, _ = v.hits()
        rays = np.repeat(np.arange(v.n_rays), np.diff(ray_off).astype(np.int64))
        x, y = rays % cams[0].width, rays // cams[0].width
        r = rect[gid]
        assert np.all((x >= r[:, 0]) & (x <= r[:, 2]) & (y >= r[:, 1]) & (y <= r[:, 3]))
        assert np.all(cls[gid] != 0)


def test_prefilter_equals_brute_force():
    sc, cams = gs.config_cluster(n=400, width=96, height=80)
    osc = orc.OracleScene.from_scene(sc)
    a, b = orc.View(osc, cams[0]), orc.View(osc, cams[0])
    assert a.find_hits(orc.BRUTE) == b.find_hits(orc.PREFILTER)
    for p, q in zip(a.hits(), b.hits()):
        assert np.array_equal(p, q)


# ------------------------------------------------------------------ tile map
@pytest.mark.parametrize("ts", [8, 16])
def test_tile_map_against_overlap_test(ts):
    sc, cams = gs.config_tiny()
    cam = cams[0]
    rect, _, _ = orc.bounds(orc.OracleScene.from_scene(sc), cam)
    tile_off, pair_gid, slots = orc.tile_map(rect, cam.width, cam.height, ts)
    tx_n, ty_n = -(-cam.width // ts), -(-cam.height // ts)
    valid = rect[:, 2] >= rect[:, 0]
    assert slots == int(((rect[:, 2] - rect[:, 0] + 1) * (rect[:, 3] - rect[:, 1] + 1))[valid].sum())
    assert np.all(np.diff(tile_off.astype(np.int64)) >= 0) and tile_off[-1] == len(pair_gid)
    total = 0
    for ty in range(ty_n):
        for tx in range(tx_n):
            ov = valid & (rect[:, 0] < (tx + 1) * ts) & (rect[:, 2] >= tx * ts) & \
                 (rect[:, 1] < (ty + 1) * ts) & (rect[:, 3] >= ty * ts)
            t = ty * tx_n + tx
            assert np.array_equal(pair_gid[tile_off[t]:tile_off[t + 1]], np.nonzero(ov)[0])  # ascending ids
            total += int(ov.sum())
    assert total == len(pair_gid)


# ------------------------------------------------------------------ maximum-response point
def test_tstar_is_the_mahalanobis_minimiser():
    rng = np.random.default_rng(4)
    sc, cams = gs.config_tiny(n=40)
    cam = gs.pinhole(64, 64, 50.0, gs.look_at((0.3, 0.2, -0.5), (0, 0, 3)))
    # unit quaternions in float64: the library rotation used below normalises its input
    q64 = sc.quat.astype(np.float64)
    q64 /= np.linalg.norm(q64, axis=1, keepdims=True)
    osc = orc.OracleScene(sc.mean, sc.scale, q64, sc.opacity, sc.sh, sc.sh_degree)
    v = orc.View(osc, cam)
    for _ in range(60):
        i = int(rng.integers(osc.n))
        ray = int(rng.integers(v.n_rays))
        o, d = orc.ray(cam, ray % 64, ray // 64)
        R = _rot(osc.quat[i])
        Sigma = R @ np.diag(osc.scale[i] ** 2) @ R.T
        Si = np.linalg.inv(Sigma)
        f = lambda t: float((o + t * d - osc.mean[i]) @ Si @ (o + t * d - osc.mean[i]))
        alpha, ts = v.eval_pair(ray, i)
        # closed form from the covariance (the benchmark's statement of t*)
        ts_ref = ((osc.mean[i] - o) @ Si @ d) / (d @ Si @ d)
        assert ts == pytest.approx(ts_ref, rel=1e-9)
        res = minimize_scalar(f, bracket=(ts - 1.0, ts + 1.0), tol=1e-12)
        assert res.fun >= f(ts) - 1e-9 * max(1.0, f(ts))
        assert res.x == pytest.approx(ts, abs=1e-5 * max(1.0, abs(ts)))
        # compare exponents: alpha itself underflows towards 1e-300 for far-off pairs
        if f(ts) < 1000.0:
            assert math.log(alpha / osc.opacity[i]) == pytest.approx(-0.5 * f(ts), rel=1e-7, abs=1e-9)
        else:
            assert alpha < 1e-200


def test_tstar_isotropic_is_closest_approach():
    sc = _one([[0.3, -0.2, 3.0]], [[0.07] * 3], [[0.5, 0.5, -0.5, 0.5]], [0.8])
    cam = gs.pinhole(32, 32, 40.0)
    v = orc.View(sc, cam)
    for ray in (0, 100, 517, 1023):
        o, d = orc.ray(cam, ray % 32, ray // 32)
        _, ts = v.eval_pair(ray, 0)
        assert ts == pytest.approx((sc.mean[0] - o) @ d, rel=1e-12)
