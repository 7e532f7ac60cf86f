"""Pins of the oracle's per-hit intermediate-buffer entries, of the channel-split conditioning of the gradient
sums, and of the 8-byte entry encoding used by the tests."""
import numpy as np

import gart_scenes as gs
import lt16
from oracle import gart_oracle as orc


def _view(sh_degree=3, bg=(0.3, 0.1, 0.6)):
    sc, cams = gs.config_tiny(sh_degree=sh_degree)
    cam = cams[0]
    sc.sh[::3, 0, 1] = -3.0          # green clamped at zero on a third of the Gaussians
    sc.sh[1::5, 0, :] = -3.0         # every channel clamped on some
    osc = orc.OracleScene.from_scene(sc)
    v = orc.View(osc, cam, bg=bg)
    assert v.find_hits() > 2000
    v.composite()
    return osc, cam, v, np.asarray(bg)


def _rays_of_hits(v, ray_off):
    return np.repeat(np.arange(v.n_rays), np.diff(ray_off).astype(np.int64))


def test_entries_follow_their_definition_by_explicit_suffix_sums():
    osc, cam, v, bg = _view()
    ray_off, gid, t, alpha = v.hits()
    entry, flags = v.lt_entries()
    assert entry.shape == (gid.size, 4) and np.all(flags <= 7) and np.any(flags != 7) and np.any(flags == 7)
    checked = 0
    for r in range(0, v.n_rays, 7):
        b, e = int(ray_off[r]), int(ray_off[r + 1])
        if e - b < 2:
            continue
        d = orc.ray(cam, r % cam.width, r // cam.width)[1]
        Y = orc.sh_basis(d)
        raw = 0.5 + np.einsum("k,hkc->hc", Y, osc.sh[gid[b:e]])
        col = np.maximum(raw, 0.0)
        T = np.concatenate([[1.0], np.cumprod(1 - alpha[b:e])])
        for i in range(e - b):
            w = T[i] * alpha[b + i]
            behind = sum(T[j] * alpha[b + j] * col[j] for j in range(i + 1, e - b)) + T[-1] * bg
            want = w * col[i] - alpha[b + i] / (1 - alpha[b + i]) * behind
            assert np.allclose(entry[b + i, :3], want, rtol=1e-10, atol=1e-14)
            assert np.isclose(entry[b + i, 3], w, rtol=1e-12)
            assert flags[b + i] == sum(int(raw[i, c] > 0) << c for c in range(3))
            checked += 1
    assert checked > 300


def test_entries_reproduce_the_opacity_and_sh_gradients():
    """alpha dL/dalpha = <g, entry.xyz>, so dL/dsigma = sum <g, xyz> / sigma; dL/dsh_k = sum Y_k w g on unclamped channels."""
    osc, cam, v, _ = _view()
    g = gs.upstream_gradient(cam, 3).astype(np.float64).reshape(-1, 3)
    grad, gabs, gelem = v.backward(g, with_abs=True, with_elem=True)
    ray_off, gid, _, _ = v.hits()
    entry, flags = v.lt_entries()
    rays = _rays_of_hits(v, ray_off)
    ad = (g[rays] * entry[:, :3]).sum(axis=1)
    dsig = np.zeros(osc.n)
    np.add.at(dsig, gid, ad / osc.opacity[gid])
    assert np.allclose(grad[:, 10], dsig, rtol=1e-10, atol=1e-14)
    K = 16
    Y = np.stack([orc.sh_basis(orc.ray(cam, r % cam.width, r // cam.width)[1]) for r in range(v.n_rays)])
    on = (flags[:, None] >> np.arange(3)[None, :]) & 1
    wch = entry[:, 3:4] * g[rays] * on                                   # [H,3]
    dsh = np.zeros((osc.n, K, 3))
    np.add.at(dsh, gid, Y[rays][:, :, None] * wch[:, None, :])
    assert np.allclose(grad[:, 11:], dsh.reshape(osc.n, -1), rtol=1e-10, atol=1e-14)
    # the channel-split conditioning of the same two sums, written out
    esig = np.zeros(osc.n)
    np.add.at(esig, gid, np.abs(g[rays] * entry[:, :3]).sum(axis=1) / osc.opacity[gid])
    assert np.allclose(gelem[:, 10], esig, rtol=1e-10, atol=1e-14)
    esh = np.zeros((osc.n, K, 3))
    np.add.at(esh, gid, np.abs(Y[rays][:, :, None] * wch[:, None, :]))
    assert np.allclose(gelem[:, 11:], esh.reshape(osc.n, -1), rtol=1e-10, atol=1e-14)
    assert np.allclose(gelem[:, 11:], gabs[:, 11:], rtol=1e-12, atol=0)


def test_channel_split_conditioning_bounds_the_plain_one():
    osc, cam, v, _ = _view(sh_degree=1)
    g = gs.upstream_gradient(cam, 5).astype(np.float64)
    grad, gabs, gelem = v.backward(g, with_abs=True, with_elem=True)
    assert np.all(gelem >= gabs * (1 - 1e-12)) and np.any(gelem[:, :11] > 1.01 * gabs[:, :11])
    # one colour channel upstream: nothing to split
    g1 = g.copy()
    g1[..., 1:] = 0.0
    grad1, gabs1, gelem1 = v.backward(g1, with_abs=True, with_elem=True)
    assert np.allclose(gelem1, gabs1, rtol=1e-12, atol=0) and np.any(gabs1[:, :11] > 0)
    # every geometry word scales with alpha dL/dalpha: the ratio of the two scales is the same for words 0..10 of a
    # Gaussian with a single hit
    ray_off, gid, _, _ = v.hits()
    single = np.nonzero(np.bincount(gid, minlength=osc.n) == 1)[0]
    for i in single[:20]:
        nz = gabs[i, :11] > 0
        ratio = gelem[i, :11][nz] / gabs[i, :11][nz]
        assert np.allclose(ratio, ratio[0], rtol=1e-9)


def test_product_split_conditioning():
    """The finest scale splits every channel's term into its two products |g| (T alpha col + alpha Rs / (1 - alpha)):
    it bounds the channel split, equals it where nothing lies behind a hit (one composited hit per ray, black
    background), and for the opacity word it is the sum written out from the weights and the entries."""
    osc, cam, v, bg = _view(sh_degree=1)
    g = gs.upstream_gradient(cam, 7).astype(np.float64)
    grad, gabs, gelem, gterms = v.backward(g, with_abs=True, with_elem=True, with_terms=True)
    assert np.all(gterms >= gelem * (1 - 1e-12)) and np.any(gterms[:, :11] > 1.05 * gelem[:, :11])
    assert np.allclose(gterms[:, 11:], gabs[:, 11:], rtol=1e-12, atol=0)
    # opacity word: sum over hits and channels of |g| (w col + (w col - entry)) / sigma, since alpha Rs / (1 - alpha) = w col - entry
    ray_off, gid, _, _ = v.hits()
    entry, flags = v.lt_entries()
    rays = _rays_of_hits(v, ray_off)
    d = np.stack([orc.ray(cam, r % cam.width, r // cam.width)[1] for r in range(v.n_rays)])
    Y = np.stack([orc.sh_basis(x) for x in d])[:, :osc.sh.shape[1]]
    col = np.maximum(0.5 + np.einsum("hk,hkc->hc", Y[rays], osc.sh[gid]), 0.0)
    wcol = entry[:, 3:4] * col
    mass = (np.abs(g.reshape(-1, 3)[rays]) * (np.abs(wcol) + np.abs(wcol - entry[:, :3]))).sum(axis=1)
    want = np.zeros(osc.n)
    np.add.at(want, gid, mass / osc.opacity[gid])
    assert np.allclose(gterms[:, 10], want, rtol=1e-9, atol=1e-14)
    # nothing behind: one composited hit per ray and a black background
    lone = orc.View(osc, cam, bg=(0.0, 0.0, 0.0), max_hits=1)
    lone.set_hits(ray_off, gid)
    lone.composite()
    _, e1, t1 = lone.backward(g, with_elem=True, with_terms=True)
    assert np.allclose(t1, e1, rtol=1e-12, atol=0) and np.any(e1[:, :11] > 0)


def test_half_entry_encoding_round_trip():
    rng = np.random.default_rng(0)
    H = 200_000
    mag = 10.0 ** rng.uniform(-9, 0.9, size=(H, 4))
    entry = mag * np.where(rng.random((H, 4)) < 0.5, -1.0, 1.0)
    entry[:, 3] = np.abs(entry[:, 3]).clip(max=1.0)
    entry[:100] = 0.0
    flags = rng.integers(0, 8, size=H).astype(np.uint8)
    words = lt16.encode(entry, flags)
    assert words.dtype == np.uint16 and words.shape == (H, 4)
    dec, f2 = lt16.decode(words)
    assert np.array_equal(f2, flags)
    assert np.all(dec[:100] == 0.0)
    x, dx = entry[:, :3], dec[:, :3]
    normal = np.abs(x) >= lt16.TINY
    assert np.all(np.abs(dx - x)[normal] <= lt16.REL_X * np.abs(x)[normal])
    assert np.all(np.abs(dx - x)[~normal] <= lt16.ABS_SUB)
    w, dw = entry[:, 3], dec[:, 3]
    nw = w >= lt16.TINY
    assert np.all(np.abs(dw - w)[nw] <= lt16.REL_W * w[nw]) and np.all(np.abs(dw - w)[~nw] <= lt16.ABS_SUB)
    assert np.all(np.sign(dx[normal]) == np.sign(x[normal])) and np.all(dw >= 0)
    # saturation instead of infinity
    big = lt16.decode(lt16.encode(np.array([[1e3, -1e3, 20.0, 1.0]]), np.array([7], np.uint8)))[0][0]
    assert np.all(np.isfinite(big)) and abs(big[0] - 60000 / 4096) < 0.02 and abs(big[1] + 60000 / 4096) < 0.02
    # ties at nine bits go to the even neighbour: 1 + 2^-10 lies halfway between 1 and 1 + 2^-9
    half = lambda v: lt16.decode(lt16.encode(np.array([[v / 4096, 0, 0, 0]]), np.array([0], np.uint8)))[0][0, 0] * 4096
    assert half(1 + 2.0 ** -10) == 1.0 and half(1 + 3 * 2.0 ** -10) == 1 + 2.0 ** -8
