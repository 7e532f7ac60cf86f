"""Pins of the oracle's narrow kernels: response exp(-D^k / 2) with an even k > 2 in place of the Gaussian of Eq. 4 (k = 2).

The paper's benchmark uses k = 2 (Sec. 5.2) and lists narrow kernels among the compromises of 3DGRT (Sec. 5.5); it gives no
formula, so the reading is: D the Mahalanobis distance of the ray's closest point (Eq. 5), alpha = sigma exp(-D^k / 2),
clamping radius (2 ln(sigma / alpha_min))^(1/k).  Pinned by a closed form for one isotropic primitive, by the projected
surface of the clamping ellipsoid, by the hits being exactly the rays with D below the clamping radius, by central
differences of every gradient word, and by k = 2 being the plain view."""
import math

import numpy as np
import pytest

import gart_scenes as gs
from oracle import gart_oracle as orc

AMIN = 1.0 / 255.0
Y0 = 0.5 / math.sqrt(math.pi)


def _scene(mean, scale, quat, opacity, sh, deg):
    n = len(opacity)
    K = (deg + 1) ** 2
    return orc.OracleScene(np.asarray(mean, float).reshape(n, 3), np.asarray(scale, float).reshape(n, 3),
                           np.asarray(quat, float).reshape(n, 4), np.asarray(opacity, float),
                           np.asarray(sh, float).reshape(n, K, 3), deg)


def _rot(q):
    w, x, y, z = q
    return np.array([[1 - 2 * (y * y + z * z), 2 * (x * y - w * z), 2 * (x * z + w * y)],
                     [2 * (x * y + w * z), 1 - 2 * (x * x + z * z), 2 * (y * z - w * x)],
                     [2 * (x * z - w * y), 2 * (y * z + w * x), 1 - 2 * (x * x + y * y)]])


@pytest.mark.parametrize("k", [2, 4, 6])
def test_single_isotropic_primitive_closed_form(k):
    """C = sigma exp(-(perp / s)^k / 2) c where that reaches alpha_min, else 0 (perp: distance of the centre from the ray)."""
    cam = gs.pinhole(48, 40, 45.0, gs.look_at((0.5, -0.3, -3.0), (0.1, 0.0, 0.0)))
    mu, s, sigma = np.array([0.2, 0.1, 0.4]), 0.35, 0.7
    dc = np.array([0.9, 0.2, -0.1])
    q = np.array([0.3, -0.5, 0.4, 0.7]); q /= np.linalg.norm(q)
    sc = _scene([mu], [[s] * 3], [q], [sigma], [dc], 0)
    out = orc.render(sc, cam, kernel_degree=k)
    D = np.zeros((cam.height, cam.width, 3))
    for y in range(cam.height):
        for x in range(cam.width):
            o, D[y, x] = orc.ray(cam, x, y)
    p = mu - o
    perp = np.sqrt(np.maximum(p @ p - (D @ p) ** 2, 0.0))
    alpha = sigma * np.exp(-0.5 * (perp / s) ** k)
    hit = (alpha >= AMIN) & ((D @ p) > 0)
    col = np.maximum(0.0, 0.5 + Y0 * dc)
    assert hit.sum() > 100 and (~hit).sum() > 100
    assert np.allclose(out["color"], np.where(hit[..., None], alpha[..., None] * col, 0.0), rtol=1e-11, atol=1e-15)
    assert np.allclose(out["t_final"], np.where(hit, 1 - alpha, 1.0), rtol=1e-12)
    assert np.array_equal(out["hit_count"], hit.astype(np.uint32))


def test_narrower_kernel_has_the_smaller_footprint_and_the_flatter_top():
    cam = gs.pinhole(64, 64, 40.0)
    sc = _scene([[0, 0, 3.0]], [[0.3, 0.2, 0.25]], [[1, 0, 0, 0]], [0.9], [[1.0, 1.0, 1.0]], 0)
    a2 = 1.0 - orc.render(sc, cam, kernel_degree=2)["t_final"]
    a4 = 1.0 - orc.render(sc, cam, kernel_degree=4)["t_final"]
    assert (a4 > 0).sum() < (a2 > 0).sum()                         # clamping radius tau^(1/4) < tau^(1/2) for tau > 1
    inner = a2 > 0.9 * math.exp(-0.5)                               # rays with D < 1: there D^4 < D^2
    outer = (a2 > 0) & ~inner
    assert inner.sum() > 10 and np.all(a4[inner] >= a2[inner]) and outer.sum() > 10 and np.all(a4[outer] <= a2[outer])


@pytest.mark.parametrize("k", [4, 6])
def test_bounds_enclose_the_projected_clamping_ellipsoid(k):
    """Surface samples of the ellipsoid of radius (2 ln(sigma / alpha_min))^(1/k), projected: the rectangle is their hull."""
    rng = np.random.default_rng(5)
    cam = gs.pinhole(640, 480, 60.0, gs.look_at((0.3, -0.2, -4.0), (0.0, 0.1, 0.0)))
    n = 40
    mean = rng.uniform(-1.0, 1.0, (n, 3))
    scale = np.exp(rng.uniform(math.log(0.03), math.log(0.4), (n, 3)))
    quat = rng.standard_normal((n, 4)); quat /= np.linalg.norm(quat, axis=1, keepdims=True)
    op = rng.uniform(0.05, 0.99, n)
    sc = _scene(mean, scale, quat, op, np.zeros((n, 1, 3)), 0)
    rect, cls, _ = orc.bounds(sc, cam, kernel_degree=k)
    rect2, _, _ = orc.bounds(sc, cam, kernel_degree=2)
    i = np.arange(100_000) + 0.5
    phi, th = np.arccos(1 - 2 * i / i.size), np.pi * (1 + 5 ** 0.5) * i
    u = np.stack([np.cos(th) * np.sin(phi), np.sin(th) * np.sin(phi), np.cos(phi)], 1)
    Rc, tc = cam.w2c[:, :3], cam.w2c[:, 3]
    exact = 0
    for j in range(n):
        ac = (2 * math.log(op[j] / AMIN)) ** (1.0 / k)
        pc = (mean[j] + (u * (scale[j] * ac)) @ _rot(quat[j]).T) @ Rc.T + tc
        assert cls[j] == 1 and pc[:, 2].min() > 0.01
        px, py = cam.fx * pc[:, 0] / pc[:, 2] + cam.cx, cam.fy * pc[:, 1] / pc[:, 2] + cam.cy
        s = [max(0, math.ceil(px.min() - 0.5)), max(0, math.ceil(py.min() - 0.5)),
             min(cam.width - 1, math.floor(px.max() - 0.5)), min(cam.height - 1, math.floor(py.max() - 0.5))]
        if s[2] < s[0] or s[3] < s[1]:
            continue
        r = rect[j]
        assert r[0] <= s[0] and r[1] <= s[1] and r[2] >= s[2] and r[3] >= s[3]
        assert s[0] - r[0] <= 1 and s[1] - r[1] <= 1 and r[2] - s[2] <= 1 and r[3] - s[3] <= 1
        exact += list(r) == s
        if 2 * math.log(op[j] / AMIN) > 1.0:                      # radius above one: the narrow kernel's footprint is smaller
            assert r[2] - r[0] <= rect2[j][2] - rect2[j][0] and r[3] - r[1] <= rect2[j][3] - rect2[j][1]
    assert exact >= 0.85 * n


def _fd_setup(k):
    rng = np.random.default_rng(11)
    n, deg = 6, 1
    K = (deg + 1) ** 2
    mean = np.concatenate([rng.uniform(-0.3, 0.3, (n, 2)), rng.uniform(2.0, 3.0, (n, 1))], 1)
    scale = np.exp(rng.uniform(math.log(0.1), math.log(0.4), (n, 3)))
    quat = rng.standard_normal((n, 4)); quat /= np.linalg.norm(quat, axis=1, keepdims=True)
    op = rng.uniform(0.3, 0.95, n)
    sh = np.concatenate([rng.uniform(0, 1, (n, 1, 3)), rng.normal(0, 0.3, (n, K - 1, 3))], 1)
    cam = gs.pinhole(12, 10, 35.0, gs.look_at((0.2, -0.1, -0.3), (0.0, 0.0, 2.5)))
    g = rng.standard_normal((cam.height, cam.width, 3))
    return dict(mean=mean, scale=scale, quat=quat, opacity=op, sh=sh), deg, cam, g


@pytest.mark.parametrize("k", [4, 6])
def test_backward_matches_central_differences(k):
    params, deg, cam, g = _fd_setup(k)
    bg = (0.2, 0.5, 0.1)

    def view(p):
        return orc.View(orc.OracleScene(p["mean"], p["scale"], p["quat"], p["opacity"], p["sh"], deg), cam, bg=bg, kernel_degree=k)

    v = view(params)
    H = v.find_hits()
    assert H > 60
    v.composite()
    grad = v.backward(g)
    ray_off, gid, _, _ = v.hits()

    def loss(p):
        w = view(p)
        w.set_hits(ray_off, gid)              # frozen hit sets and order
        return float((w.composite()[0] * g).sum())

    K = (deg + 1) ** 2
    for name, base, width in [("mean", 0, 3), ("scale", 3, 3), ("quat", 6, 4), ("opacity", 10, 1), ("sh", 11, 3 * K)]:
        flat = params[name].reshape(params[name].shape[0], -1)
        for i in range(flat.shape[0]):
            for j in range(width):
                x0 = flat[i, j]
                h = 1e-3 if name == "sh" else 1e-6 * max(abs(x0), 0.1)
                flat[i, j] = x0 + h; lp = loss(params)
                flat[i, j] = x0 - h; lm = loss(params)
                flat[i, j] = x0
                fd, an = (lp - lm) / (2 * h), grad[i, base + j]
                assert abs(fd - an) / max(abs(an), abs(fd), 1e-3) < 5e-6, (name, i, j, fd, an)


def test_degree_two_is_the_plain_view_and_the_hits_are_the_rays_inside_the_clamping_radius():
    sc, cams = gs.config_tiny(n=120, sh_degree=1, width=32, height=24, seed=4)
    sc.scale *= np.float32(2.0)
    osc, cam = orc.OracleScene.from_scene(sc), cams[0]
    g = gs.upstream_gradient(cam, 1).astype(np.float64)
    a = orc.render(osc, cam, dL_dC=g)
    b = orc.render(osc, cam, dL_dC=g, kernel_degree=2)
    assert np.array_equal(a["color"], b["color"]) and np.allclose(a["grad"], b["grad"], rtol=1e-12, atol=1e-14)   # (threads sum in any order)
    # k = 4: alpha of every listed hit equals sigma exp(-D^4 / 2) with D^2 = -2 ln(alpha_2 / sigma) of the same pair at k = 2
    v4 = orc.View(osc, cam, kernel_degree=4)
    v4.find_hits(orc.BRUTE)
    ray_off, gid, _, alpha4 = v4.hits()
    rays = np.repeat(np.arange(cam.width * cam.height), np.diff(ray_off).astype(np.int64))
    v2 = orc.View(osc, cam)
    for h in range(0, gid.size, 7):
        a2, _ = v2.eval_pair(int(rays[h]), int(gid[h]))
        D2 = -2.0 * math.log(a2 / osc.opacity[gid[h]])
        assert abs(alpha4[h] - osc.opacity[gid[h]] * math.exp(-0.5 * D2 * D2)) <= 1e-12
        assert alpha4[h] >= AMIN
