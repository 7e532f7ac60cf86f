"""Pins for the oracle's compositing (Eq. 6-8) and analytic backward.

Closed forms, invariants and finite differences; no expected value is produced
by the function under test.
"""
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


def _rays(cam):
    o = None
    D = np.zeros((cam.height, cam.width, 3))
    for y in range(cam.height):
        for x in range(cam.width):
            o, D[y, x] = orc.ray(cam, x, y)
    return o, D


def test_single_isotropic_gaussian_closed_form():
    """C = sigma exp(-(|mu-o|^2 - ((mu-o).d)^2) / (2 s^2)) c where that is >= alpha_min, else 0; T_final = 1 - alpha."""
    cam = gs.pinhole(48, 40, 45.0, gs.look_at((0.5, -0.3, -3.0), (0.1, 0.0, 0.0)))
    mu, s, sigma = np.array([0.2, 0.1, 0.4]), 0.35, 0.7
    dc = np.array([0.9, 0.2, -0.1])                      # DC coefficients; colour = 0.5 + Y0 * dc
    # an isotropic Gaussian is rotation invariant only for orthogonal R: use a unit quaternion
    q = np.array([0.3, -0.5, 0.4, 0.7]); q /= np.linalg.norm(q)
    sc = _scene([mu], [[s] * 3], [q], [sigma], [dc], 0)
    out = orc.render(sc, cam)
    o, D = _rays(cam)
    p = mu - o
    perp2 = p @ p - (D @ p) ** 2
    alpha = sigma * np.exp(-perp2 / (2 * s * s))
    hit = (alpha >= AMIN) & ((D @ p) > 0)
    col = np.maximum(0.0, 0.5 + Y0 * dc)
    ref = np.where(hit[..., None], alpha[..., None] * col, 0.0)
    assert hit.sum() > 100 and (~hit).sum() > 100
    assert np.allclose(out["color"], ref, rtol=1e-12, atol=1e-15)
    assert np.allclose(out["t_final"], np.where(hit, 1 - alpha, 1.0), rtol=1e-12)
    assert np.array_equal(out["hit_count"], hit.astype(np.uint32))


def test_behind_camera_maximum_is_not_a_hit():
    cam = gs.pinhole(16, 16, 60.0)
    sc = _scene([[0, 0, -0.5]], [[1.0, 1.0, 1.0]], [[1, 0, 0, 0]], [0.9], [[1, 1, 1]], 0)
    out = orc.render(sc, cam, near=-10.0)     # even if the near rule lets it through, t* < 0 rejects it
    assert out["hit_count"].sum() == 0 and np.all(out["color"] == 0) and np.all(out["t_final"] == 1)


def test_transmittance_product_and_partition_of_unity():
    sc, cams = gs.config_tiny()
    kappa = 0.37
    sh = np.full((sc.n, 1, 3), (kappa - 0.5) / Y0)
    osc = orc.OracleScene(sc.mean, sc.scale, sc.quat, sc.opacity, sh, 0)
    v = orc.View(osc, cams[0], bg=(kappa, kappa, kappa))
    v.find_hits()
    color, t_final, cnt = v.composite()
    ray_off, gid, t, alpha = v.hits()
    assert cnt.max() >= 5
    for r in range(v.n_rays):
        a = alpha[ray_off[r]:ray_off[r + 1]]
        assert t_final.reshape(-1)[r] == pytest.approx(np.prod(1 - a), rel=1e-13)
        assert np.all(np.diff(t[ray_off[r]:ray_off[r + 1]]) >= 0)
    assert np.allclose(color, kappa, rtol=1e-13)             # sum T_i alpha_i + T_final = 1
    v2 = orc.View(osc, cams[0])
    v2.find_hits()
    c2, tf2, _ = v2.composite()
    assert np.allclose(c2, kappa * (1 - tf2)[..., None], rtol=1e-12, atol=1e-15)


def test_two_gaussians_order_by_tstar_and_permutation_invariance():
    """Two needles whose centre depths and t* disagree in order on part of the image."""
    cam = gs.pinhole(40, 40, 50.0)
    th = math.radians(70.0)                                  # long axis tilted strongly towards the viewer
    qa = [math.cos(th / 2), 0.0, math.sin(th / 2), 0.0]
    mean = [[-0.05, 0.0, 3.0], [0.05, 0.0, 3.1]]
    scale = [[0.5, 0.05, 0.02], [0.5, 0.05, 0.02]]
    quat = [qa, [math.cos(-th / 2), 0.0, math.sin(-th / 2), 0.0]]
    op = [0.8, 0.6]
    sh = [[[1.2, -0.4, 0.3]], [[-0.6, 0.9, 1.5]]]
    sc = _scene(mean, scale, quat, op, sh, 0)
    out = orc.render(sc, cam)
    v = out["view"]
    ray_off, gid, t, alpha = v.hits()
    col = np.maximum(0.0, 0.5 + Y0 * np.array(sh).reshape(2, 3))
    both = swapped = 0
    for r in range(v.n_rays):
        a0, t0 = v.eval_pair(r, 0)
        a1, t1 = v.eval_pair(r, 1)
        h0, h1 = a0 >= AMIN and t0 > 0, a1 >= AMIN and t1 > 0
        if h0 and h1:
            first, second = (0, 1) if (t0, 0) < (t1, 1) else (1, 0)
            af, as_ = (a0, a1) if first == 0 else (a1, a0)
            ref = af * col[first] + (1 - af) * as_ * col[second]
            both += 1
            swapped += first == 1
        elif h0 or h1:
            ref = (a0 if h0 else a1) * col[0 if h0 else 1]
        else:
            ref = np.zeros(3)
        assert np.allclose(out["color"].reshape(-1, 3)[r], ref, rtol=1e-12, atol=1e-15)
    assert both > 20 and 0 < swapped < both                   # both orders occur although z(0) < z(1)
    perm = [1, 0]
    sc2 = _scene(np.array(mean)[perm], np.array(scale)[perm], np.array(quat)[perm], np.array(op)[perm],
                 np.array(sh)[perm], 0)
    assert np.allclose(orc.render(sc2, cam)["color"], out["color"], rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------ backward
def _fd_scene(deg):
    rng = np.random.default_rng(7)
    n = 7
    K = (deg + 1) ** 2
    mean = np.concatenate([rng.uniform(-0.35, 0.35, (n, 2)), rng.uniform(2.0, 3.0, (n, 1))], 1)
    scale = np.exp(rng.uniform(math.log(0.08), math.log(0.4), (n, 3)))
    quat = rng.standard_normal((n, 4))
    quat /= np.linalg.norm(quat, axis=1, keepdims=True)
    op = rng.uniform(0.3, 0.95, n)
    sh = np.concatenate([rng.uniform(0, 1, (n, 1, 3)), rng.normal(0, 0.3, (n, K - 1, 3))], 1)
    sh[0, 0, :] = -9.0        # one Gaussian with all channels clamped at zero
    sh[1, 0, 1] = -9.0        # one with a single clamped channel
    cam = gs.pinhole(12, 10, 35.0, gs.look_at((0.2, -0.1, -0.3), (0.0, 0.0, 2.5)))
    g = rng.standard_normal((cam.height, cam.width, 3))
    return dict(mean=mean, scale=scale, quat=quat, opacity=op, sh=sh), deg, cam, g


def _loss(params, deg, cam, g, lists, bg):
    sc = orc.OracleScene(params["mean"], params["scale"], params["quat"], params["opacity"], params["sh"], deg)
    v = orc.View(sc, cam, bg=bg)
    v.set_hits(*lists)                       # frozen hit sets and order: the loss is smooth in every parameter
    color, _, _ = v.composite()
    return float((color * g).sum())


@pytest.mark.parametrize("deg", [0, 3])
def test_backward_matches_central_differences(deg):
    params, deg, cam, g = _fd_scene(deg)
    bg = (0.2, 0.5, 0.1)
    sc = orc.OracleScene(params["mean"], params["scale"], params["quat"], params["opacity"], params["sh"], deg)
    v = orc.View(sc, cam, bg=bg)
    H = v.find_hits()
    color, _, cnt = v.composite()
    assert H > 200 and cnt.max() >= 4
    grad = v.backward(g)
    ray_off, gid, _, _ = v.hits()
    lists = (ray_off, gid)
    K = (deg + 1) ** 2
    layout = [("mean", 0, 3), ("scale", 3, 3), ("quat", 6, 4), ("opacity", 10, 1), ("sh", 11, 3 * K)]
    worst = 0.0
    for name, base, width in layout:
        arr = params[name]
        flat = arr.reshape(arr.shape[0], -1)
        for i in range(flat.shape[0]):
            for j in range(width):
                x0 = flat[i, j]
                # the loss is piecewise linear in the SH coefficients: a wide step is exact there
                h = 1e-3 if name == "sh" else 1e-6 * max(abs(x0), 0.1)
                flat[i, j] = x0 + h
                lp = _loss(params, deg, cam, g, lists, bg)
                flat[i, j] = x0 - h
                lm = _loss(params, deg, cam, g, lists, bg)
                flat[i, j] = x0
                fd = (lp - lm) / (2 * h)
                an = grad[i, base + j]
                err = abs(fd - an) / max(abs(an), abs(fd), 1e-3)
                worst = max(worst, err)
                assert err < 2e-6, (name, i, j, fd, an)
    # clamped colour channels carry no SH gradient
    assert np.all(grad[0, 11:] == 0) and np.all(grad[1, 11 + 1::3] == 0) and np.any(grad[1, 11::3] != 0)


def test_backward_invariants():
    sc, cams = gs.config_tiny()
    cam = cams[0]
    sc.mean[0] = (50.0, 0.0, 3.0)       # off screen
    sc.opacity[1] = 0.001               # below alpha_min
    sc.mean[2] = (0.0, 0.0, -3.0)       # behind the camera
    osc = orc.OracleScene.from_scene(sc)
    g = gs.upstream_gradient(cam, 0).astype(np.float64)
    v = orc.View(osc, cam)
    v.find_hits()
    color, t_final, cnt = v.composite()
    grad, gabs = v.backward(g, with_abs=True)
    ray_off, gid, t, alpha = v.hits()
    # (a) Gaussians without hits have exactly zero gradient
    hit_any = np.zeros(osc.n, bool)
    hit_any[gid] = True
    assert (~hit_any).sum() == 3 and np.all(grad[~hit_any] == 0) and np.any(grad[hit_any] != 0)
    assert np.all(gabs >= np.abs(grad) * (1 - 1e-12))
    # (b) linear in the upstream gradient
    # (threads add in varying order, so compare against the conditioning of each sum)
    assert np.all(np.abs(v.backward(2.5 * g) - 2.5 * grad) <= 1e-12 * gabs)
    # (c) degree-0 DC gradient = Y0 * sum over hits of T_i alpha_i g (all colours unclamped here)
    T = np.zeros_like(alpha)
    for r in range(v.n_rays):
        a = alpha[ray_off[r]:ray_off[r + 1]]
        T[ray_off[r]:ray_off[r + 1]] = np.concatenate([[1.0], np.cumprod(1 - a)[:-1]])
    rays = np.repeat(np.arange(v.n_rays), np.diff(ray_off).astype(np.int64))
    ref = np.zeros((osc.n, 3))
    np.add.at(ref, gid, Y0 * (T * alpha)[:, None] * g.reshape(-1, 3)[rays])
    assert np.all(0.5 + Y0 * osc.sh[:, 0, :] > 0)
    assert np.allclose(grad[:, 11:14], ref, rtol=1e-11, atol=1e-14)
    # (d) opacity gradient, written out: sum g.(T c - R/(1-alpha)) * alpha/sigma, with R by explicit suffix sums
    col = np.maximum(0.0, 0.5 + Y0 * osc.sh[:, 0, :])
    dsig = np.zeros(osc.n)
    for r in range(v.n_rays):
        b, e = int(ray_off[r]), int(ray_off[r + 1])
        for h in range(b, e):
            R = sum(T[j] * alpha[j] * col[gid[j]] for j in range(h + 1, e))
            dal = g.reshape(-1, 3)[r] @ (T[h] * col[gid[h]] - R / (1 - alpha[h]))
            dsig[gid[h]] += dal * alpha[h] / osc.opacity[gid[h]]
    assert np.allclose(grad[:, 10], dsig, rtol=1e-10, atol=1e-13)


def test_translation_invariance_sum_dmu_equals_minus_dorigin():
    """Moving every Gaussian by delta equals moving the camera by -delta: sum_i dL/dmu_i = -dL/do (by differences)."""
    params, deg, cam, g = _fd_scene(0)
    sc = orc.OracleScene(params["mean"], params["scale"], params["quat"], params["opacity"], params["sh"], deg)
    v = orc.View(sc, cam)
    v.find_hits()
    v.composite()
    grad = v.backward(g)
    lists = v.hits()[:2]
    R, t = cam.w2c[:, :3], cam.w2c[:, 3]
    o = -R.T @ t
    for ax in range(3):
        vals = []
        for sgn in (+1, -1):
            o2 = o.copy()
            o2[ax] += sgn * 1e-6
            w2c = np.concatenate([R, (-R @ o2)[:, None]], 1)
            cam2 = gs.Camera(cam.width, cam.height, cam.fx, cam.fy, cam.cx, cam.cy, w2c)
            v2 = orc.View(sc, cam2)
            v2.set_hits(*lists)
            c2, _, _ = v2.composite()
            vals.append(float((c2 * g).sum()))
        dLdo = (vals[0] - vals[1]) / 2e-6
        assert grad[:, ax].sum() == pytest.approx(-dLdo, rel=1e-5, abs=1e-7)
