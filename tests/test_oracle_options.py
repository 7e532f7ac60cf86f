"""Pins of the oracle's optional compromises (early termination at a transmittance threshold, alpha clamp -- the
shortcuts that the paper's comparison with 3DGRT lists and its own benchmark switches off, Sec. 5.2 / 5.5) and of its
conditioning measure for single-precision transmittances.

Early termination is pinned against hit lists cut by hand at the position a numpy prefix product finds (a path that
knows nothing of the option); the clamp against a numpy re-compositing of the clamped alphas, against central
differences, and by the structural fact that a clamped hit passes no gradient through alpha; the conditioning against
brute-force perturbation of every alpha of a ray in an explicit numpy restatement of the entries."""
import numpy as np
import pytest

import gart_scenes as gs
from oracle import gart_oracle as orc


def _scene(seed=6, deg=2, n=300, opaque=False):
    sc, cams = gs.config_tiny(n=n, sh_degree=deg, width=28, height=22, seed=seed)
    sc.scale *= np.float32(3.0)          # a dozen hits per ray on this small image
    if opaque:
        rng = np.random.default_rng(seed)
        sc.opacity[:] = np.where(rng.random(sc.n) < 0.3, rng.uniform(0.99, 0.9995, sc.n), sc.opacity).astype(np.float32)
    return sc, cams[0], orc.OracleScene.from_scene(sc)


def _colours(osc, cam, ray_off, gid):
    rays = np.repeat(np.arange(cam.width * cam.height), np.diff(ray_off).astype(np.int64))
    Y = np.stack([orc.sh_basis(orc.ray(cam, r % cam.width, r // cam.width)[1]) for r in range(cam.width * cam.height)])
    raw = 0.5 + np.einsum("hk,hkc->hc", Y[rays][:, :osc.sh.shape[1]], osc.sh[gid])
    return rays, np.maximum(raw, 0.0), Y


@pytest.mark.parametrize("t_min", [0.5, 0.1, 0.01])
def test_early_termination_equals_hand_cut_lists(t_min):
    sc, cam, osc = _scene()
    bg = (0.2, 0.6, 0.1)
    g = gs.upstream_gradient(cam, 2).astype(np.float64)
    full = orc.View(osc, cam, bg=bg)
    full.find_hits()
    ray_off, gid, _, alpha = full.hits()
    # where each ray ends: before the first hit whose transmittance in front is below t_min (plain prefix products)
    keep = np.zeros(cam.width * cam.height, np.int64)
    for r in range(keep.size):
        b, e = int(ray_off[r]), int(ray_off[r + 1])
        T = np.concatenate([[1.0], np.cumprod(1.0 - alpha[b:e])])[:e - b]
        below = np.nonzero(T < t_min)[0]
        keep[r] = below[0] if below.size else e - b
    assert (keep < np.diff(ray_off)).sum() > 20 and keep.max() > 3
    new_off = np.zeros(ray_off.size, np.uint64)
    new_off[1:] = np.cumsum(keep)
    idx = np.concatenate([np.arange(int(ray_off[r]), int(ray_off[r]) + int(keep[r])) for r in range(keep.size)])
    cut = orc.View(osc, cam, bg=bg)
    cut.set_hits(new_off, gid[idx])
    c2, t2, _ = cut.composite()
    g2, a2 = cut.backward(g, with_abs=True)

    term = orc.View(osc, cam, bg=bg, t_min=t_min)
    term.set_hits(ray_off, gid)
    c1, t1, n1 = term.composite()
    g1, a1 = term.backward(g, with_abs=True)
    assert np.array_equal(c1, c2) and np.array_equal(t1, t2)
    assert np.array_equal(n1.reshape(-1), np.diff(ray_off).astype(np.uint32))     # the lists still hold every hit
    assert np.all(np.abs(g1 - g2) <= 1e-12 * np.maximum(a1, a2))
    e1, _ = term.lt_entries()
    dropped = np.ones(gid.size, bool)
    dropped[idx] = False
    assert dropped.any() and np.all(e1[dropped] == 0.0)
    # every ray that ended early did so with T_final below the threshold, the others above it
    ended = keep < np.diff(ray_off)
    assert np.all(t1.reshape(-1)[ended] < t_min) and np.all(t1.reshape(-1)[~ended & (np.diff(ray_off) > 0)] >= 0.0)
    m_t, m_a = term.margins()
    assert 0.0 < m_t < 10.0 and m_a == np.inf
    # t_min = 0 is the plain view
    c0, t0, _ = full.composite()
    assert np.abs(c0 - c1).max() > 1e-4 and np.all(t1 >= t0 - 1e-15)


def test_alpha_clamp_composites_the_clamped_alphas():
    sc, cam, osc = _scene(seed=8, opaque=True)
    bg = np.array([0.1, 0.3, 0.5])
    a_max = 0.9
    v = orc.View(osc, cam, bg=tuple(bg), alpha_max=a_max)
    v.find_hits()
    ray_off, gid, _, alpha = v.hits()
    assert (alpha > a_max).sum() > 50
    color, t_final, _ = v.composite()
    rays, col, Y = _colours(osc, cam, ray_off, gid)
    ae = np.minimum(alpha, a_max)
    for r in range(0, cam.width * cam.height, 3):
        b, e = int(ray_off[r]), int(ray_off[r + 1])
        T = np.concatenate([[1.0], np.cumprod(1.0 - ae[b:e])])
        want = (T[:-1, None] * ae[b:e, None] * col[b:e]).sum(axis=0) + T[-1] * bg
        assert np.allclose(color.reshape(-1, 3)[r], want, rtol=1e-12, atol=1e-15)
        assert np.isclose(t_final.reshape(-1)[r], T[-1], rtol=1e-12)
    entry, flags = v.lt_entries()
    assert np.all(entry[alpha > a_max, :3] == 0.0) and np.all(entry[alpha > a_max, 3] > 0.0)
    m_t, m_a = v.margins()
    assert m_t == np.inf and 0.0 < m_a < 1.0


def test_alpha_clamp_gradient_by_central_differences():
    """With fixed hit lists L = sum <g, C> is differentiable wherever no alpha sits on the clamp: compare the analytic
    gradient with central differences of the oracle's own compositing on a few Gaussians, some of whose hits are clamped."""
    sc, cam, osc = _scene(seed=9, n=60, deg=1, opaque=True)
    a_max = 0.95
    g = gs.upstream_gradient(cam, 4).astype(np.float64)
    base = orc.View(osc, cam, alpha_max=a_max)
    base.find_hits()
    lists = base.hits()[:2]
    base.composite()
    assert base.margins()[1] > 1e-4
    grad = base.backward(g)
    _, gid, _, alpha = base.hits()
    clamped_g = np.unique(gid[alpha > a_max])
    assert clamped_g.size > 3

    def loss(scene_arrays):
        o2 = orc.OracleScene(*scene_arrays, sc.sh_degree)
        v = orc.View(o2, cam, alpha_max=a_max)
        v.set_hits(*lists)
        c, _, _ = v.composite()
        return float((g * c).sum())

    arrays = [osc.mean, osc.scale, osc.quat, osc.opacity, osc.sh]
    word0 = [0, 3, 6, 10, 11]
    checked = 0
    for i in list(clamped_g[:3]) + [int(x) for x in np.setdiff1d(np.unique(gid), clamped_g)[:2]]:
        for a, w0 in zip(range(5), word0):
            flat = arrays[a].reshape(osc.n, -1)
            for j in range(min(flat.shape[1], 4)):
                h = 1e-6 * max(1.0, abs(flat[i, j]))
                keep = flat[i, j]
                flat[i, j] = keep + h; lp = loss(arrays)
                flat[i, j] = keep - h; lm = loss(arrays)
                flat[i, j] = keep
                fd = (lp - lm) / (2 * h)
                assert abs(fd - grad[i, w0 + j]) <= 2e-6 * max(1.0, abs(fd)) + 1e-8, (i, a, j, fd, grad[i, w0 + j])
                checked += 1
    assert checked > 50
    # a Gaussian all of whose hits are clamped gets a gradient only through its colour (a clamp low enough to have such)
    low = orc.View(osc, cam, alpha_max=0.01)
    low.set_hits(*lists)
    low.composite()
    grad_low = low.backward(g)
    all_cl = [i for i in np.unique(gid) if np.all(alpha[gid == i] > 0.01)]
    some_free = [i for i in np.unique(gid) if np.any(alpha[gid == i] < 0.01)]
    assert len(all_cl) >= 2 and some_free
    for i in all_cl:
        assert np.all(grad_low[i, :11] == 0.0) and np.any(grad_low[i, 11:] != 0.0)
    assert any(np.any(grad_low[i, :11] != 0.0) for i in some_free)


def _entries_numpy(alpha, col, bg):
    """Entries of one ray written out from their definition (Eq. 6-8): prefix products and suffix sums."""
    n = alpha.size
    T = np.concatenate([[1.0], np.cumprod(1.0 - alpha)])
    w = T[:-1] * alpha
    out = np.zeros((n, 4))
    for i in range(n):
        B = (w[i + 1:, None] * col[i + 1:]).sum(axis=0) + T[-1] * bg
        out[i, :3] = w[i] * col[i] - alpha[i] / (1.0 - alpha[i]) * B
        out[i, 3] = w[i]
    return out


def test_conditioning_bounds_every_alpha_perturbation():
    """cond of the entries: perturb every alpha of a ray by a relative eps with arbitrary signs; to first order no word
    moves by more than eps x cond, and a perturbation of one sign comes within a small factor of the bound."""
    sc, cam, osc = _scene(seed=11, opaque=True, n=400)
    bg = np.array([0.4, 0.2, 0.3])
    v = orc.View(osc, cam, bg=tuple(bg))
    v.find_hits()
    v.composite()
    ray_off, gid, _, alpha = v.hits()
    entry, flags, cond = v.lt_entries(with_cond=True)
    rays, col, _ = _colours(osc, cam, ray_off, gid)
    assert np.all(cond >= np.abs(entry) * (1 - 1e-12))                 # (the word itself is part of its conditioning)
    rng = np.random.default_rng(3)
    eps = 1e-7
    worst = 0.0
    tested = 0
    for r in range(0, cam.width * cam.height, 5):
        b, e = int(ray_off[r]), int(ray_off[r + 1])
        if e - b < 4:
            continue
        base = _entries_numpy(alpha[b:e], col[b:e], bg)
        assert np.allclose(base, entry[b:e], rtol=1e-9, atol=1e-15)
        for trial in range(6):
            s = np.ones(e - b) if trial == 0 else (-np.ones(e - b) if trial == 1 else rng.choice([-1.0, 1.0], e - b))
            moved = _entries_numpy(alpha[b:e] * (1.0 + eps * s), col[b:e], bg)
            d = np.abs(moved - base)
            bound = eps * cond[b:e] * (1.0 + 1e-3) + 1e-6 * eps * np.abs(base).max() + 1e-18   # (second-order terms: eps^2 kappa^2)
            assert np.all(d <= bound), (r, trial, float((d / np.maximum(bound, 1e-300)).max()))
            nz = cond[b:e] > 1e-12
            worst = max(worst, float((d[nz] / (eps * cond[b:e][nz])).max()))
        tested += 1
    assert tested > 30 and worst > 0.3          # the bound is met to within a small factor: it is not vacuous
    # rays with a nearly opaque hit in front are the ill-conditioned ones
    kappa_like = cond[:, 3] / np.maximum(entry[:, 3], 1e-300)
    assert kappa_like.max() > 100.0 and kappa_like.min() >= 1.0 - 1e-12


def test_gradient_conditioning_written_out_from_the_entries():
    sc, cam, osc = _scene(seed=12, opaque=True, deg=1)
    v = orc.View(osc, cam, bg=(0.2, 0.2, 0.2))
    v.find_hits()
    v.composite()
    g = gs.upstream_gradient(cam, 6).astype(np.float64).reshape(-1, 3)
    grad, gabs, gcond = v.backward(g, with_abs=True, with_cond=True)
    ray_off, gid, _, _ = v.hits()
    entry, flags, cond = v.lt_entries(with_cond=True)
    rays, col, Y = _colours(osc, cam, ray_off, gid)
    # opacity word: sum over hits of sum_c |g_c| cond_c / sigma
    want = np.zeros(osc.n)
    np.add.at(want, gid, (np.abs(g[rays]) * cond[:, :3]).sum(axis=1) / osc.opacity[gid])
    assert np.allclose(gcond[:, 10], want, rtol=1e-9, atol=1e-15)
    # SH words: sum over hits of |Y_k g_c| cond_w on the unclamped channels
    K = osc.sh.shape[1]
    on = (flags[:, None] >> np.arange(3)[None, :]) & 1
    wsh = np.zeros((osc.n, K, 3))
    np.add.at(wsh, gid, np.abs(Y[rays][:, :K, None] * (cond[:, 3:4] * g[rays] * on)[:, None, :]))
    assert np.allclose(gcond[:, 11:], wsh.reshape(osc.n, -1), rtol=1e-9, atol=1e-15)
    # and it dominates the plain mass of the terms (kappa >= 0)
    assert np.all(gcond >= gabs * (1 - 1e-9))
