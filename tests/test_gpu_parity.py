"""GPU parity: the CUDA path (through the C ABI) against the float64 oracle, element by element.

Tolerances (each fp32 term carries a relative error of a few 1e-6, so a sum is off by about 1e-5 of the mass of its
terms whatever the summation order):
  * rectangles, classes, tile offsets, pair lists, per-ray hit counts and ordered hit lists:
    bit-exact, up to the guard-band protocol of tests/parity.py;
  * colour: |gpu - ref| <= 1e-4 |ref| + 1e-7; final transmittance: 1e-4 |ref| + 1e-6;
  * gradients (all 11+3K words, every backward variant): |gpu - ref| <= 1e-3 max(|ref|, COND * A)
    or <= 1e-6, where A is the mass of the fp32 products that the word is summed from (its conditioning): per hit
    the absolute contribution, with alpha dL/dalpha = sum_c g_c (T alpha col_c - alpha Rs_c / (1 - alpha)) counted
    as sum_c |g_c| (|T alpha col_c| + |alpha Rs_c / (1 - alpha)|) -- a hit whose colour is close to the colour behind it
    cancels inside one term.  A sum whose terms cancel to less than COND = 2% of their mass cannot reach a
    relative 1e-3 in fp32 in any summation order, so the relative bar is measured against that floor;
    plus EPS_ALPHA * K, where K is the oracle's first-order effect on the word of a unit relative error of every alpha on
    the word's rays (through the transmittances: a hit with alpha close to 1 in front multiplies the error of its own
    alpha by alpha / (1 - alpha) in everything behind it, which no fp32 path avoids) and EPS_ALPHA = 3e-6 bounds the
    relative error of an alpha evaluated in single precision (an exponential of a quadratic form of rounded inputs: a few
    ulp of 6e-8 each from the form, the exponential and the product);
  * gradients from 8-byte LT entries (lt_format 2): the same bar plus 1.05 * 2^-10 * E, where E is the sum of
    the absolute per-hit terms split by colour channel.  Every gradient word is linear in the four words of the
    hit's entry, each stored to a relative 2^-10 (2^-11 for the weight), so that is the bound of the encoding;
    the entries themselves are compared with the oracle's (tests/parity.py: check_lt16).
"""
import dataclasses

import numpy as np
import pytest
import torch

import gart_scenes as gs
import paper_2608_17298_b200.gart as G
from oracle import gart_oracle as orc

import parity as P

pytestmark = pytest.mark.gpu

COND = 0.02
EPS_ALPHA = 3e-6


def assert_color(gpu, ref, sel, cam):
    dc, ac, dt, at = P.color_errors(gpu, ref, sel, cam)
    assert np.all(dc <= 1e-4 * ac + 1e-7), float((dc / np.maximum(ac, 1e-30)).max())
    assert np.all(dt <= 1e-4 * at + 1e-6)


def assert_grad(gpu_grad, ref, K, rows=None):
    gw = 11 + 3 * K
    rows = np.arange(ref["grad"].shape[0]) if rows is None else rows
    g = gpu_grad[rows][:, :gw].astype(np.float64)
    r, a, kc = ref["grad"][rows], ref["gterms"][rows], ref["gcond"][rows]
    d = np.abs(g - r)
    ok = (d <= 1e-3 * np.maximum(np.abs(r), COND * a) + EPS_ALPHA * kc) | (d <= 1e-6)
    assert ok.all(), ("gradient outside tolerance", int((~ok).sum()), float(d[~ok].max()))
    assert np.all(gpu_grad[rows][:, gw:] == 0)
    strict = (d <= 1e-3 * np.abs(r)) | (d <= 1e-6)
    return float(strict.mean())


def assert_grad_lt16(gpu_grad, ref, K, rows=None):
    gw = 11 + 3 * K
    rows = np.arange(ref["grad"].shape[0]) if rows is None else rows
    gpu_grad = gpu_grad[rows]
    g = gpu_grad[:, :gw].astype(np.float64)
    r, a, e = ref["grad"][rows], ref["gterms"][rows], ref["gelem"][rows]
    d = np.abs(g - r)
    ok = d <= 1.05 * 2.0 ** -10 * e + np.maximum(1e-3 * np.maximum(np.abs(r), COND * a), 1e-6)
    assert ok.all(), ("gradient from 8-byte entries outside tolerance", int((~ok).sum()), float(d[~ok].max()))
    assert np.all(gpu_grad[:, gw:] == 0)
    # the encoding costs precision but not much: most words stay within 0.3 % of the oracle's
    return float(((d <= 3e-3 * np.maximum(np.abs(r), COND * a)) | (d <= 1e-6)).mean())


VARIANTS = ("grad", "grad_tile", "grad_atomic", "grad_atomic_vec", "grad_hybrid", "grad_warp")   # every backward pass on 16-byte (4-byte: hybrid) entries


OPTION_BAND = 1e-3    # rays with a termination or clamp decision closer than this (in ln) to its threshold carry no upstream gradient


def option_band(scene, cam, cfg):
    """Rays on which a decision of the options t_min / alpha_max comes within OPTION_BAND of flipping under float64:
    |ln(T_i / t_min)| or |ln(alpha / alpha_max)| below the band.  Each option puts one more floating-point comparison on
    the compositing path; on these rays single precision may take it the other way, which changes the ray's colour and its
    hits' entries by a whole term.  The tests give such rays a zero upstream gradient and leave their colour unchecked (at
    most a few per thousand); on every other ray the decisions are then required to be the oracle's."""
    v = orc.View(orc.OracleScene.from_scene(scene), cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32, max_hits=cfg.max_hits,
                 t_min=cfg.t_min_f32, alpha_max=cfg.alpha_max_f32 if cfg.alpha_max < 1.0 else 1.0, kernel_degree=cfg.kernel_degree)
    v.find_hits()
    v.composite()
    return (v.ray_margins() < OPTION_BAND).any(axis=1)


def full_parity(scene, cam, cfg, g=None, mode=orc.BRUTE, guard=False, caps=(None, None)):
    g = gs.upstream_gradient(cam, 0) if g is None else g
    keep = np.ones(cam.width * cam.height, bool)
    if cfg.t_min > 0 or cfg.alpha_max < 1:
        keep = ~option_band(scene, cam, cfg)
        assert keep.mean() > 0.99
        g = (np.asarray(g).reshape(-1, 3) * keep[:, None]).reshape(np.asarray(g).shape).astype(np.float32)
    gpu = P.run_gpu(scene, cam, cfg, g, cap_pairs=caps[0], cap_hits=caps[1], guard=guard)
    assert gpu["counts"][G.CNT_ERROR] == 0
    m = P.check_maps(scene, cam, cfg, gpu)
    P.check_structure(cam, cfg, gpu)
    P.check_structure_tile(cam, cfg, gpu)
    ref = P.check_hits_and_replay(m["osc"], cam, cfg, gpu, g, None, mode)
    assert ref["view"].ray_margins()[keep].min(initial=np.inf) > 0.1 * OPTION_BAND   # (the replayed lists are the GPU's: a guard-band hit may move a margin a little)
    ref["keep"] = keep
    assert_color(gpu, ref, ref["sel"][keep], cam)
    K = (scene.sh_degree + 1) ** 2
    strict = {v: assert_grad(gpu[v], ref, K) for v in VARIANTS if v in gpu}
    assert min(strict.values()) > 0.995, strict            # the conditioning floor is the exception, not the rule
    ref["lt32_worst"] = P.check_lt32(gpu, ref, keep)
    P.check_lt16(gpu, ref, keep)
    assert assert_grad_lt16(gpu["grad_lt16"], ref, K) > 0.85
    ref["strict"] = strict
    return gpu, ref


# ------------------------------------------------------------------------------------------ small configs, every ray
@pytest.mark.parametrize("ts", [8, 16])
def test_tiny_exact_lists_and_values(ts):
    scene, cams = gs.config_tiny()
    gpu, ref = full_parity(scene, cams[0], G.Config(tile_size=ts))
    st = ref["stats"]
    assert st["identical_lists"] and st["band_hit"] == 0 and st["band_order"] == 0   # no guard-band case at all on Tiny
    assert gpu["counts"][G.CNT_HITS] == st["oracle_hits"]


@pytest.mark.parametrize("deg", [0, 1, 2, 3])
def test_tiny_all_sh_degrees(deg):
    scene, cams = gs.config_tiny(sh_degree=deg, seed=deg + 1)
    full_parity(scene, cams[0], G.Config(tile_size=8))


@pytest.mark.parametrize("ts", [8, 16])
def test_cluster10k_every_ray(ts):
    scene, cams = gs.config_cluster()
    gpu, ref = full_parity(scene, cams[0], G.Config(tile_size=ts))
    assert ref["stats"]["band_hit"] + ref["stats"]["band_order"] <= 1e-4 * ref["stats"]["oracle_hits"]


@pytest.mark.parametrize("m", [1, 6])
def test_hit_cap(m):
    """Only the first m hits of every ray are composited: colour, T_final, LT entries and every gradient follow
    the oracle's capped compositing; lists, counts and slots still describe all hits."""
    scene, cams = gs.config_cluster(n=4000, width=120, height=96, seed=21)
    cam = cams[0]
    gpu, ref = full_parity(scene, cam, G.Config(max_hits=m, background=(0.1, 0.3, 0.2)))
    free, _ = full_parity(scene, cam, G.Config(background=(0.1, 0.3, 0.2)))
    assert np.array_equal(gpu["ray_gid"], free["ray_gid"]) and np.array_equal(gpu["hit_count"], free["hit_count"])
    assert gpu["hit_count"].max() > 3 * m
    assert np.abs(gpu["color"] - free["color"]).max() > 1e-2 and np.all(gpu["t_final"] >= free["t_final"] - 1e-6)
    # Gaussians that only ever lie behind the cap get a zero gradient
    first = np.zeros(scene.n, bool)
    ro = gpu["ray_off"].astype(np.int64)
    for r in range(ro.size - 1):
        first[gpu["ray_gid"][ro[r]:min(ro[r] + m, ro[r + 1])]] = True
    hidden = ~first & (np.bincount(gpu["ray_gid"], minlength=scene.n) > 0)
    assert hidden.any() and np.all(gpu["grad"][hidden] == 0) and np.all(gpu["grad_atomic"][hidden] == 0) and np.all(gpu["grad_tile"][hidden] == 0)


@pytest.mark.parametrize("seed", [101, 102, 103, 104, 105, 106])
def test_random_configurations(seed):
    """Random combinations of image size (ragged against both tile sizes), field of view, SH degree, tile size, background,
    alpha_min, hit cap, early termination, alpha clamp and kernel degree on a random cluster, every ray and every backward variant against the oracle."""
    rng = np.random.default_rng(seed)
    deg = int(rng.integers(0, 4))
    width, height = int(rng.integers(40, 150)), int(rng.integers(30, 110))
    scene, cams = gs.config_cluster(n=int(rng.integers(500, 5000)), sh_degree=deg, width=width, height=height, seed=seed)
    # a camera somewhere around the cluster (centre (0, 0, 3)), looking near its centre, any field of view
    dirv = rng.normal(size=3)
    pos = np.array([0.0, 0.0, 3.0]) + float(rng.uniform(2.0, 4.0)) * dirv / np.linalg.norm(dirv)
    cam = gs.pinhole(width, height, float(rng.uniform(25.0, 75.0)), gs.look_at(pos, np.array([0.0, 0.0, 3.0]) + rng.uniform(-0.2, 0.2, 3)))
    cfg = G.Config(tile_size=int(rng.choice([8, 16])), background=tuple(float(v) for v in rng.uniform(0, 1, 3)),
                   alpha_min=float(rng.choice([1.0 / 255.0, 0.01, 0.03])), max_hits=int(rng.choice([0, 0, 3, 17])))
    cfg.t_min, cfg.alpha_max = float(rng.choice([0.0, 0.0, 0.03, 0.2])), float(rng.choice([1.0, 1.0, 0.95, 0.6]))
    cfg.kernel_degree = int(np.random.default_rng([seed, 7]).choice([2, 2, 4]))   # (a stream of its own: the other draws stay what they were)
    gpu, ref = full_parity(scene, cam, cfg, g=gs.upstream_gradient(cam, seed))
    assert gpu["counts"][G.CNT_HITS] > 100


@pytest.mark.parametrize("seed", [3, 11, 19, 42])
def test_random_cameras_inside_the_cloud(seed):
    """Harsher random scenes: scales from sub-pixel needles to screen-filling blobs, the camera inside or beside the
    cloud (Gaussians behind it, straddling its plane, covering the image), fy != fx and an off-centre principal point."""
    rng = np.random.default_rng(seed)
    deg = int(rng.integers(0, 4))
    n = int(rng.integers(50, 1500))
    width, height = int(rng.integers(17, 120)), int(rng.integers(9, 100))
    mean = rng.uniform(-1.0, 1.0, (n, 3))
    scale = np.exp(rng.uniform(np.log(0.003), np.log(0.6), (n, 3)))
    scene = gs.Scene(mean.astype(np.float32), scale.astype(np.float32), gs._unit_quats(rng, n).astype(np.float32),
                     gs._sigmoid(rng.normal(0, 2.0, n)).astype(np.float32), gs._sh(rng, n, deg), deg)
    cam = gs.pinhole(width, height, float(rng.uniform(20.0, 100.0)), gs.look_at(rng.uniform(-1.5, 1.5, 3), rng.uniform(-0.5, 0.5, 3)))
    cam = gs.Camera(cam.width, cam.height, cam.fx, cam.fx * float(rng.uniform(0.8, 1.25)), cam.cx + float(rng.uniform(-5, 5)),
                    cam.cy + float(rng.uniform(-5, 5)), cam.w2c)
    cfg = G.Config(tile_size=int(rng.choice([8, 16])), background=tuple(float(v) for v in rng.uniform(0, 1, 3)),
                   alpha_min=float(rng.choice([1.0 / 255.0, 0.02])), max_hits=int(rng.choice([0, 0, 0, 5])))
    gpu, ref = full_parity(scene, cam, cfg, g=gs.upstream_gradient(cam, seed))
    assert gpu["counts"][G.CNT_HITS] > 0


def test_early_termination():
    """t_min: a ray ends before the first hit with less than t_min transmittance in front of it; colour, T_final, LT
    entries and every gradient follow the oracle's early-terminated compositing; lists and counts still hold every hit."""
    scene, cams = gs.config_cluster(n=4000, width=120, height=96, seed=23)
    cam = cams[0]
    t_min = 0.05
    gpu, ref = full_parity(scene, cam, G.Config(t_min=t_min, background=(0.2, 0.1, 0.3)))
    free, _ = full_parity(scene, cam, G.Config(background=(0.2, 0.1, 0.3)))
    keep = ref["keep"].reshape(cam.height, cam.width)
    assert not keep.all()                                           # (the band is met on a view of this size: the protocol is exercised)
    assert np.array_equal(gpu["ray_gid"], free["ray_gid"]) and np.array_equal(gpu["hit_count"], free["hit_count"])
    ended = gpu["t_final"] < t_min
    assert 0.05 < ended.mean() < 0.95
    assert np.all(gpu["t_final"] >= free["t_final"] - 1e-6) and np.abs(gpu["color"] - free["color"]).max() > 1e-3
    same = ~ended & (free["t_final"] >= 1.01 * t_min)              # rays that never meet the threshold are untouched, to the bit
    assert same.any() and np.array_equal(gpu["color"][same], free["color"][same])


def test_alpha_clamp():
    """alpha_max: every hit composites min(alpha, alpha_max); a clamped hit passes no gradient through alpha."""
    scene, cams = gs.config_cluster(n=4000, width=120, height=96, seed=24)
    scene.opacity[::3] = np.float32(0.97)
    cam = cams[0]
    a_max = 0.9
    gpu, ref = full_parity(scene, cam, G.Config(alpha_max=a_max))
    free, _ = full_parity(scene, cam, G.Config())
    assert np.abs(gpu["color"] - free["color"]).max() > 1e-3 and np.all(gpu["t_final"] >= free["t_final"] - 1e-7)
    # both options with a cap, on the tile-major passes too (full_parity runs every variant)
    full_parity(scene, cam, G.Config(alpha_max=a_max, max_hits=9, tile_size=16))


@pytest.mark.parametrize("ts", [8, 16])
def test_narrow_kernel(ts):
    """kernel_degree = 4: response exp(-D^4 / 2).  Rectangles (clamping radius tau^(1/4)), hit lists, colour, LT entries and the
    gradients of every backward pass that takes the option follow the oracle's; the footprints shrink, the hybrid pass refuses."""
    scene, cams = gs.config_cluster(n=4000, width=120, height=96, seed=27)
    cam = cams[0]
    cfg = G.Config(kernel_degree=4, tile_size=ts, background=(0.1, 0.2, 0.3))
    gpu, ref = full_parity(scene, cam, cfg)
    free, _ = full_parity(scene, cam, G.Config(tile_size=ts, background=(0.1, 0.2, 0.3)))
    assert 0 < gpu["counts"][G.CNT_PAIRS] < free["counts"][G.CNT_PAIRS] and 0 < gpu["counts"][G.CNT_HITS] < free["counts"][G.CNT_HITS]
    assert np.abs(gpu["color"] - free["color"]).max() > 1e-3
    assert "grad_hybrid" not in gpu and "grad_hybrid" in free
    # with the options of the other compromises too
    full_parity(scene, cam, G.Config(kernel_degree=4, tile_size=ts, alpha_max=0.9, max_hits=12))


@pytest.mark.parametrize("ts", [8, 16])
def test_no_write_outside_any_buffer(ts):
    """Every device buffer of the view sits between two guard zones; after the whole path in every variant (both LT
    layouts, three entry formats, five backward passes) with the capacities at their exact need, the zones are untouched."""
    scene, cams = gs.config_cluster(n=3000, width=150, height=90, seed=31)
    cfg = G.Config(tile_size=ts)
    g = G.Gaussians.from_numpy(scene)
    pairs, _ = G.size_view(cfg, g, cams[0], slack=1.0)
    probe = P.run_gpu(scene, cams[0], cfg, gs.upstream_gradient(cams[0], 0))
    need = max(int(probe["counts"][G.CNT_LT_SLOTS]), int(probe["tile"]["lt_slots"]))     # (the larger of the two layouts' needs)
    full_parity(scene, cams[0], cfg, guard=True, caps=(pairs - 1, need))
    # one entry short: the forward reports it and writes nothing outside
    short = P.run_gpu(scene, cams[0], cfg, gs.upstream_gradient(cams[0], 0), cap_pairs=pairs - 1, cap_hits=need - 1, atomic=False, guard=True)
    assert short["counts"][G.CNT_ERROR] != 0


def test_stricter_alpha_min():
    """alpha_min is a parameter (the paper's 1/255 is the default): a stricter threshold drops hits on both sides alike."""
    scene, cams = gs.config_cluster(n=4000, width=120, height=96, seed=22)
    gpu, ref = full_parity(scene, cams[0], G.Config(alpha_min=0.05))
    free, _ = full_parity(scene, cams[0], G.Config())
    assert 0 < gpu["counts"][G.CNT_HITS] < 0.8 * free["counts"][G.CNT_HITS]


def test_ragged_image_and_background():
    scene, cams = gs.config_tiny(width=61, height=37, sh_degree=2, seed=5)
    for ts in (8, 16):
        full_parity(scene, cams[0], G.Config(tile_size=ts, background=(0.2, 0.5, 0.1)))


def test_forward_without_ray_lists_gives_the_same_view():
    """The per-ray ordered lists are optional outputs: without them colour, T_final, LT and the gradient are the
    same bits (the lists only serve the pixel-centric baseline and the parity checks)."""
    scene, cams = gs.config_cluster(n=3000, width=96, height=80, seed=11)
    cam, cfg = cams[0], G.Config()
    g = G.Gaussians.from_numpy(scene)
    dl = torch.from_numpy(gs.upstream_gradient(cam, 0)).cuda()
    cap_pairs, cap_hits = G.size_view(cfg, g, cam, slack=1.0)
    outs = []
    for lists in (True, False):
        buf = G.ViewBuffers(g.n, g.sh_degree, cam, cfg, cap_pairs, cap_hits)
        buf.ray_gid.fill_(-1)
        G.run_bounds_tile_map(cfg, g, cam, buf)
        G.run_forward(cfg, g, cam, buf, ray_lists=lists)
        G.run_backward(cfg, g, cam, buf, dl)
        torch.cuda.synchronize()
        cnt = G.gart_read_counts(buf.counts)
        assert cnt[G.CNT_ERROR] == 0 and cnt[G.CNT_HITS] > 0
        outs.append((buf.color.cpu().numpy().copy(), buf.t_final.cpu().numpy().copy(),
                     buf.lt.cpu().numpy()[:cnt[G.CNT_LT_SLOTS]].copy(), buf.ray_gid.cpu().numpy().copy(), cnt))
        grad = buf.grad.cpu().numpy()[:g.n]
        outs[-1] += (grad.copy(),)
    a, b = outs
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and list(a[4]) == list(b[4])
    # LT entries are written once each (padding is never written: compare the written ones through the gradient)
    # the reductions add in a different order from run to run: equal up to rounding of cancelling sums
    assert np.all(np.abs(a[5] - b[5]) <= 1e-3 * np.abs(a[5]) + 1e-6 * np.abs(a[5]).max(axis=0, keepdims=True) + 1e-9)
    assert np.all(b[3] == -1) and np.any(a[3] != -1)               # the list was left untouched


def test_straddling_gaussian_and_culling_rules():
    scene, cams = gs.config_tiny(n=64, seed=9)
    scene.mean[0] = (0.05, -0.02, 0.3); scene.scale[0] = (0.4, 0.5, 0.45); scene.opacity[0] = 0.6   # crosses the camera plane
    scene.mean[1] = (9.0, 0.0, 0.2); scene.scale[1] = (0.3, 0.3, 0.3)                              # straddles, outside the frustum
    scene.mean[2] = (0.0, 0.0, -2.0)                                                                 # behind
    scene.opacity[3] = 0.003                                                                          # below alpha_min
    scene.mean[4] = (30.0, 0.0, 3.0)                                                                  # off screen
    gpu, ref = full_parity(scene, cams[0], G.Config(tile_size=8))
    assert list(gpu["cls"][:5]) == [2, 2, 0, 0, 1]
    assert list(gpu["rect"][0]) == [0, 0, 63, 63] and list(gpu["rect"][1]) == [0, 0, -1, -1]
    assert gpu["counts"][G.CNT_STRADDLE] == 2
    assert np.any(gpu["grad"][0] != 0) and np.all(gpu["grad"][1:5] == 0)


def test_rays_longer_than_the_shared_memory_sort():
    """More than 1024 hits on a ray: the per-ray sort falls back to global memory."""
    rng = np.random.default_rng(3)
    n = 1400
    mean = np.stack([rng.normal(0, 0.02, n), rng.normal(0, 0.02, n), rng.uniform(2.0, 6.0, n)], 1)
    scene = gs.Scene(mean.astype(np.float32), np.full((n, 3), 0.25, np.float32) * rng.uniform(0.8, 1.2, (n, 3)).astype(np.float32),
                     gs._unit_quats(rng, n).astype(np.float32), rng.uniform(0.01, 0.03, n).astype(np.float32),
                     gs._sh(rng, n, 1), 1)
    cam = gs.pinhole(16, 16, 20.0)
    gpu, ref = full_parity(scene, cam, G.Config(tile_size=8))
    assert gpu["counts"][G.CNT_MAX_RAY_HITS] > 1024
    capped, _ = full_parity(scene, cam, G.Config(tile_size=8, max_hits=700))   # the cap on that path
    assert np.abs(capped["color"] - gpu["color"]).max() > 1e-5


@pytest.mark.parametrize("deg", [0, 1, 2, 3])
def test_many_rank_groups_and_multi_chunk_pairs(deg):
    """Hundreds of pairs per tile, every pair hitting (almost) all 64 pixels: each warp of the backward walks
    several rank groups and several LT chunks per group, re-using its shared-memory buffers every time."""
    rng = np.random.default_rng(11 + deg)
    n = 400
    mean = np.stack([rng.normal(0, 0.02, n), rng.normal(0, 0.02, n), rng.uniform(2.0, 6.0, n)], 1)
    scene = gs.Scene(mean.astype(np.float32), np.full((n, 3), 0.25, np.float32) * rng.uniform(0.8, 1.2, (n, 3)).astype(np.float32),
                     gs._unit_quats(rng, n).astype(np.float32), rng.uniform(0.01, 0.03, n).astype(np.float32),
                     gs._sh(rng, n, deg), deg)
    cam = gs.pinhole(16, 16, 20.0)
    for rep in range(3):          # a race would not fail every time
        full_parity(scene, cam, G.Config(tile_size=8), g=gs.upstream_gradient(cam, rep))


def test_primitive_and_atomic_backward_agree():
    scene, cams = gs.config_cluster(n=3000, width=128, height=96)
    g = gs.upstream_gradient(cams[0], 1)
    gpu = P.run_gpu(scene, cams[0], G.Config(tile_size=8), g)
    a, b = gpu["grad"].astype(np.float64), gpu["grad_atomic"].astype(np.float64)
    scale = np.maximum(np.abs(a), np.abs(b))
    close = np.abs(a - b) <= 1e-3 * scale + 1e-5 * np.abs(a).max(axis=1, keepdims=True) + 1e-6
    assert close.all()


# ------------------------------------------------------------------------------------------ full-size configs, sampled
def sampled_parity(scene, cam, cfg, view_seed, n_gauss=300, n_tiles=60, max_area=3000, n_large=20, large_max_area=40000):
    """Full-size view on the GPU; the oracle handles a sample: random tiles plus every pixel of the
    rectangles of randomly chosen Gaussians, so that those Gaussians' gradients are complete.  Two strata of
    Gaussians: rectangles of up to max_area pixels, and n_large larger ones (the background Gaussians that cover
    hundreds of tiles and are cut into many work items)."""
    g = gs.upstream_gradient(cam, view_seed)
    gpu = P.run_gpu(scene, cam, cfg, g, atomic=True)
    assert gpu["counts"][G.CNT_ERROR] == 0
    m = P.check_maps(scene, cam, cfg, gpu)
    st = P.check_structure(cam, cfg, gpu)
    P.check_structure_tile(cam, cfg, gpu)
    rng = np.random.default_rng([view_seed, 77])
    rect = gpu["rect"]
    area = (rect[:, 2] - rect[:, 0] + 1) * (rect[:, 3] - rect[:, 1] + 1)
    visible = rect[:, 2] >= rect[:, 0]
    cand = np.nonzero(visible & (area <= max_area))[0]
    gsel = rng.choice(cand, size=min(n_gauss, cand.size), replace=False)
    big = np.nonzero(visible & (area > max_area) & (area <= large_max_area))[0]
    gbig = rng.choice(big, size=min(n_large, big.size), replace=False)
    gsel = np.concatenate([gsel, gbig])
    mask = np.zeros((cam.height, cam.width), np.uint8)
    for i in gsel:
        x0, y0, x1, y1 = rect[i]
        mask[y0:y1 + 1, x0:x1 + 1] = 1
    ts = 8
    for _ in range(n_tiles):
        ty, tx = int(rng.integers(-(-cam.height // ts))), int(rng.integers(-(-cam.width // ts)))
        mask[ty * ts:(ty + 1) * ts, tx * ts:(tx + 1) * ts] = 1
    ref = P.check_hits_and_replay(m["osc"], cam, cfg, gpu, g, mask, orc.PREFILTER)
    stats = ref["stats"]
    assert stats["oracle_hits"] > 1000
    band = (stats["band_hit"] + stats["band_order"]) / stats["oracle_hits"]
    assert band <= 1e-4, stats                                        # guard-band cases: at most 1e-4 of the sampled hits
    assert_color(gpu, ref, ref["sel"], cam)
    K = (scene.sh_degree + 1) ** 2
    strict = {v: assert_grad(gpu[v], ref, K, gsel) for v in VARIANTS}
    assert min(strict.values()) >= 0.995, strict                     # share of words inside the plain 1e-3 | 1e-6 bar
    assert assert_grad_lt16(gpu["grad_lt16"], ref, K, gsel) > 0.85      # the backward on 8-byte LT entries
    print("sampled parity: %d rays, %d oracle hits, %d Gaussians (%d large); guard band: %d hit + %d order cases = %.1e of the hits; "
          "strict share %s; items %d, whole Gaussians %.3f, LT padding %.3f" % (
              stats["rays"], stats["oracle_hits"], gsel.size, gbig.size, stats["band_hit"], stats["band_order"], band,
              {k: round(v, 5) for k, v in strict.items()}, st["items"], st["whole_share"], st["lt_padding"]))
    # the prefilter of the oracle is audited by true all-pairs brute force on a few rays
    audit = np.zeros_like(mask)
    ys, xs = np.nonzero(mask)
    pick = rng.choice(ys.size, size=min(24, ys.size), replace=False)
    audit[ys[pick], xs[pick]] = 1
    va = orc.View(m["osc"], cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32)
    va.find_hits(orc.BRUTE, audit)
    vb = orc.View(m["osc"], cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32)
    vb.find_hits(orc.PREFILTER, audit)
    for p, q in zip(va.hits(), vb.hits()):
        assert np.array_equal(p, q)
    return gpu, ref


@pytest.mark.parametrize("view", [0, 1, 2, 3])
def test_shell200k_sampled(view):
    scene, cams = gs.config_shell()
    sampled_parity(scene, cams[view], G.Config(tile_size=8), view)


def test_unbounded1m_sampled():
    scene, cams = gs.config_unbounded_1m()
    sampled_parity(scene, cams[0], G.Config(tile_size=8), 0, n_gauss=200, n_tiles=40, n_large=14)
    sampled_parity(scene, cams[0], G.Config(tile_size=16), 1, n_gauss=60, n_tiles=12, n_large=6)


@pytest.mark.parametrize("view", [5, 0, 9, 12])
def test_unbounded6m_sampled(view):
    """The benchmark's configuration, in the launch configuration bench.py times (8x8 tiles): four views of the orbit,
    the first with the larger sample."""
    scene, cams = gs.config_unbounded_6m()
    if view == 5:
        gpu, ref = sampled_parity(scene, cams[view], G.Config(tile_size=8), view, n_gauss=200, n_tiles=40, n_large=12, large_max_area=20000)
    else:
        gpu, ref = sampled_parity(scene, cams[view], G.Config(tile_size=8), view, n_gauss=80, n_tiles=16, n_large=4, large_max_area=15000)
    assert gpu["counts"][G.CNT_HITS] > 1e8


def test_unbounded6m_whole_orbit_layouts_agree():
    """Every one of the benchmark's 16 views, without the oracle: the view's invariants (hit totals, transmittances in [0, 1],
    finite colours and gradients, no error word, every gradient record written) and agreement of the two decompositions of
    the backward pass, whose forward passes lay the intermediate buffer out differently: identical hit counts, colours and
    transmittances, gradients equal up to the rounding of differently ordered sums.  Compared on the device."""
    import dataclasses
    scene, cams = gs.config_unbounded_6m()
    g = G.Gaussians.from_numpy(scene)
    cfg_t = G.Config(tile_size=8, lt_layout=G.LT_TILE_MAJOR)
    cfg_p = dataclasses.replace(cfg_t, lt_layout=G.LT_PRIMITIVE_MAJOR)
    cap_pairs, cap_hits = 0, 0
    for cam in (cams[0], cams[8]):
        for cfg in (cfg_t, cfg_p):
            P, S = G.size_view(cfg, g, cam, slack=1.3)
            cap_pairs, cap_hits = max(cap_pairs, P), max(cap_hits, S)
    buf = G.ViewBuffers(g.n, g.sh_degree, cams[0], cfg_t, cap_pairs, cap_hits)
    gt, gp = torch.empty_like(buf.grad), torch.empty_like(buf.grad)
    worst = 0.0
    for v, cam in enumerate(cams):
        dl = torch.from_numpy(gs.upstream_gradient(cam, v)).cuda()
        outs = []
        for cfg, grad, back in ((cfg_t, gt, G.run_backward_tile), (cfg_p, gp, G.run_backward)):
            grad.fill_(float("nan"))
            G.run_bounds_tile_map(cfg, g, cam, buf)
            G.run_forward(cfg, g, cam, buf, ray_lists=False)
            back(cfg, g, cam, buf, dl, grad)
            cnt = G.gart_read_counts(buf.counts)
            assert cnt[G.CNT_ERROR] == 0, (v, cnt)
            assert int(buf.hit_count.view(torch.int32).sum(dtype=torch.int64)) == cnt[G.CNT_HITS] > 1e8
            assert bool(torch.isfinite(buf.color).all()) and bool(torch.isfinite(grad).all())
            assert float(buf.t_final.min()) >= 0.0 and float(buf.t_final.max()) <= 1.0
            outs.append((buf.color.clone(), buf.t_final.clone(), buf.hit_count.clone(), cnt[G.CNT_HITS], cnt[G.CNT_PAIRS]))
        a, b = outs
        assert a[3] == b[3] and a[4] == b[4] and torch.equal(a[2], b[2])
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])          # both layouts composite the very same numbers
        x, y = gt[:, :59].double(), gp[:, :59].double()
        tol = 1e-3 * torch.maximum(x.abs(), y.abs()) + 1e-5 * x.abs().amax(dim=1, keepdim=True) + 1e-6
        bad = (x - y).abs() > tol
        assert not bool(bad.any()), (v, int(bad.sum()))
        worst = max(worst, float(((x - y).abs() / tol).max()))
    print("whole orbit: 16 views, largest difference between the two backward decompositions %.2f of the tolerance" % worst)


# ------------------------------------------------------------------------------------------ edge cases and errors
def _empty_scene(deg=1):
    K = (deg + 1) ** 2
    z = lambda *s: np.zeros(s, np.float32)
    return gs.Scene(z(0, 3), z(0, 3), z(0, 4), z(0), z(0, K, 3), deg)


def test_no_gaussians():
    cam = gs.pinhole(40, 24, 50.0)
    cfg = G.Config(tile_size=8, background=(0.3, 0.1, 0.7))
    gpu = P.run_gpu(_empty_scene(), cam, cfg, gs.upstream_gradient(cam, 0), cap_pairs=0, cap_hits=0, atomic=False)
    c = gpu["counts"]
    assert c[G.CNT_PAIRS] == 0 and c[G.CNT_HITS] == 0 and c[G.CNT_ERROR] == 0
    assert np.all(gpu["tile_off"] == 0) and np.all(gpu["hit_count"] == 0)
    assert np.allclose(gpu["color"], np.array([0.3, 0.1, 0.7], np.float32)) and np.all(gpu["t_final"] == 1)


def test_everything_culled():
    scene, cams = gs.config_tiny(n=50)
    scene.opacity[:] = 0.002
    gpu = P.run_gpu(scene, cams[0], G.Config(), gs.upstream_gradient(cams[0], 0), atomic=True)
    assert gpu["counts"][G.CNT_VISIBLE] == 0 and gpu["counts"][G.CNT_PAIRS] == 0 and gpu["counts"][G.CNT_HITS] == 0
    assert np.all(gpu["grad"] == 0) and np.all(gpu["grad_atomic"] == 0) and np.all(gpu["color"] == 0)
    assert np.all(gpu["cls"] == 0) and np.all(gpu["rect"] == np.array([0, 0, -1, -1]))


def test_capacity_errors_are_reported_not_fatal():
    scene, cams = gs.config_tiny()
    cam, cfg = cams[0], G.Config()
    g = gs.upstream_gradient(cam, 0)
    gpu = P.run_gpu(scene, cam, cfg, g, cap_pairs=100, cap_hits=20000, atomic=False)
    assert gpu["counts"][G.CNT_ERROR] & 1 and gpu["counts"][G.CNT_PAIRS] == 683 and np.all(gpu["tile_off"] == 0)
    gpu = P.run_gpu(scene, cam, cfg, g, cap_pairs=700, cap_hits=500, atomic=False)
    assert gpu["counts"][G.CNT_ERROR] == 2 and gpu["counts"][G.CNT_HITS] == 7373
    # and the context is still usable afterwards
    gpu = P.run_gpu(scene, cam, cfg, g, atomic=False)
    assert gpu["counts"][G.CNT_ERROR] == 0 and gpu["counts"][G.CNT_HITS] == 7373


@pytest.mark.parametrize("variant", ["primitive", "tile", "hybrid"])
def test_a_wait_that_gives_up_is_reported_and_leaves_the_context_usable(variant):
    """wait_polls < 0: every wait of the streaming kernel for its own copies gives up without a poll.  The call returns,
    the time-out bit is set and gart_sync_status says so; the view run again on the same buffers with the normal limit gives
    the oracle's gradients.  Nothing faults and nothing hangs: the waits that give up are the kernel's own bounded ones."""
    scene, cams = gs.config_tiny()
    cam = cams[0]
    cfg = {"primitive": G.Config(lt_layout=G.LT_PRIMITIVE_MAJOR), "tile": G.Config(lt_layout=G.LT_TILE_MAJOR),
           "hybrid": G.Config(lt_layout=G.LT_TILE_MAJOR, lt_format=1)}[variant]
    fn = {"primitive": G.run_backward, "tile": G.run_backward_tile, "hybrid": G.run_backward_hybrid}[variant]
    g = G.Gaussians.from_numpy(scene)
    pairs, slots = G.size_view(cfg, g, cam)
    buf = G.ViewBuffers(g.n, g.sh_degree, cam, cfg, pairs, slots)
    dl_np = gs.upstream_gradient(cam, 0)
    dl = torch.from_numpy(np.ascontiguousarray(dl_np, dtype=np.float32)).cuda()

    def view(c):
        G.run_bounds_tile_map(c, g, cam, buf)
        G.run_forward(c, g, cam, buf)
        buf.grad.fill_(float("nan"))
        fn(c, g, cam, buf, dl)
        return G.gart_sync_status(buf.counts)

    assert view(dataclasses.replace(cfg, wait_polls=-1)) == 5                       # GART_ERR_TIMEOUT
    assert G.gart_read_counts(buf.counts)[G.CNT_ERROR] == 4                         # GART_ERRBIT_TIMEOUT alone
    assert view(dataclasses.replace(cfg, wait_polls=1 << 20)) == G.GART_OK          # (an explicit limit)
    assert view(cfg) == G.GART_OK
    got = buf.grad.cpu().numpy()[:g.n]
    ref = orc.render(orc.OracleScene.from_scene(scene), cam, dL_dC=dl_np, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32)
    K = (scene.sh_degree + 1) ** 2
    assert np.allclose(got[:, :11 + 3 * K], ref["grad"], rtol=2e-3, atol=2e-5)


def test_invalid_arguments_return_status():
    scene, cams = gs.config_tiny(n=8)
    cam = cams[0]
    g = G.Gaussians.from_numpy(scene)
    buf = G.ViewBuffers(g.n, 0, cam, G.Config(), 100, 1000)
    args = (buf.slot_of_gid, buf.gid_of_slot, buf.counts)
    with pytest.raises(G.GartError) as e:
        G.gart_bounds(G.Config(tile_size=12), g, cam, buf.rect, buf.cls, buf.pre, *args, buf.workspace)
    assert e.value.status == 1
    with pytest.raises(G.GartError) as e:
        G.gart_bounds(G.Config(), g, cam, None, buf.cls, buf.pre, *args, buf.workspace)
    assert e.value.status == 1
    with pytest.raises(G.GartError) as e:
        G.gart_bounds(G.Config(), g, cam, buf.rect, buf.cls, buf.pre, *args, buf.workspace[:512])
    assert e.value.status == 2
    G.gart_bounds(G.Config(), g, cam, buf.rect, buf.cls, buf.pre, *args, buf.workspace)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(G.GartError) as e:
        G.gart_tile_map(G.Config(), buf.rect, g.n, cam, buf.tile_off, buf.pair_gid, 100, buf.counts, small)
    assert e.value.status == 2
    with pytest.raises(G.GartError) as e:
        G.gart_tile_map(G.Config(), buf.rect, g.n, cam, buf.tile_off, buf.pair_gid, 100, buf.counts, buf.workspace[1:])
    assert e.value.status == 1                     # workspace not 256-byte aligned
    # each backward variant wants its own LT format, and the forward knows three
    dl = torch.zeros((cam.height, cam.width, 3), dtype=torch.float32, device="cuda")
    TM, PM = G.LT_TILE_MAJOR, G.LT_PRIMITIVE_MAJOR
    refused = [
        (G.run_backward, G.Config(lt_format=1, lt_layout=PM)),        # the item pass reads 16-byte entries ...
        (G.run_backward, G.Config(lt_format=2, lt_layout=PM)),
        (G.run_backward, G.Config(lt_format=1, lt_layout=TM)),        # ... the block-per-tile pass 16- or 8-byte entries
        (G.run_backward_tile, G.Config(lt_layout=PM)),                # the tile-major passes want the tile-major layout
        (G.run_backward_tile, G.Config(lt_format=1, lt_layout=TM)),
        (G.run_backward_warp, G.Config(lt_layout=PM)),
        (G.run_backward_warp, G.Config(lt_format=1, lt_layout=TM)),
        (G.run_backward_warp, G.Config(lt_format=2, lt_layout=TM)),
        (G.run_backward_hybrid, G.Config(lt_format=2, lt_layout=TM)),
        (G.run_backward_hybrid, G.Config(lt_format=1, lt_layout=PM)),
        (G.run_backward_hybrid, G.Config(lt_format=1, lt_layout=TM, max_hits=4)),
        (G.run_backward_hybrid, G.Config(lt_format=1, lt_layout=TM, t_min=0.01)),
        (G.run_backward_hybrid, G.Config(lt_format=1, lt_layout=TM, alpha_max=0.99)),
        (G.run_backward_hybrid, G.Config(lt_format=0, lt_layout=TM)),
        (G.run_backward_hybrid, G.Config(lt_format=1, lt_layout=TM, kernel_degree=4)),   # its pixel pass knows the Gaussian response only
        (G.run_backward_tile, G.Config(kernel_degree=3)),             # the library builds the degrees 2 and 4
        (G.run_backward, G.Config(lt_layout=PM, kernel_degree=6)),
    ]
    for fn, cfg_bad in refused:
        with pytest.raises(G.GartError) as e:
            fn(cfg_bad, g, cam, buf, dl)
        assert e.value.status == 1, (fn.__name__, cfg_bad)
    for cfg_bad in (G.Config(max_hits=-1), G.Config(lt_format=3), G.Config(lt_layout=2), G.Config(lt_format=1, lt_layout=G.LT_PRIMITIVE_MAJOR),
                    G.Config(lt_format=2, lt_layout=G.LT_PRIMITIVE_MAJOR),
                    G.Config(t_min=1.0), G.Config(t_min=-0.1), G.Config(alpha_max=0.0), G.Config(kernel_degree=3)):   # (refused by gart_forward)
        with pytest.raises(G.GartError) as e:
            G.run_forward(cfg_bad, g, cam, buf)
        assert e.value.status == 1, cfg_bad
    # the evaluation copies rows of SH coefficients from the caller's array in 16-byte pieces: an array that is not 16-byte
    # aligned is refused on the host
    import dataclasses
    skew = torch.zeros(g.sh.numel() + 1, dtype=torch.float32, device="cuda")[1:].view(g.sh.shape)
    with pytest.raises(G.GartError) as e:
        G.run_forward(G.Config(), dataclasses.replace(g, sh=skew), cam, buf)
    assert e.value.status == 1
    # pointers that a pass dereferences: refused on the host instead of faulting on the device
    with pytest.raises(G.GartError) as e:     # the pixel-centric baseline without the per-ray lists
        G.gart_backward_atomic(G.Config(), g, cam, buf.pre, buf.slot_of_gid, buf.ray_off, None, None, buf.lt, dl, buf.grad, buf.counts)
    assert e.value.status == 1
    with pytest.raises(G.GartError) as e:     # no intermediate buffer
        G.gart_backward(G.Config(), g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view, buf.cap_pairs, None, dl,
                        buf.grad, buf.counts, buf.workspace)
    assert e.value.status == 1
    with pytest.raises(G.GartError) as e:     # no view block
        G.gart_backward(G.Config(), g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, None, buf.cap_pairs, buf.lt, dl,
                        buf.grad, buf.counts, buf.workspace)
    assert e.value.status == 1
    with pytest.raises(G.GartError) as e:     # a view block laid out for fewer pairs
        G.gart_backward(G.Config(), g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view, buf.cap_pairs * 100, buf.lt, dl,
                        buf.grad, buf.counts, buf.workspace)
    assert e.value.status == 2
    with pytest.raises(G.GartError) as e:     # hybrid without the ray id list
        G.gart_backward_hybrid(G.Config(lt_format=1, lt_layout=TM), g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view,
                               buf.cap_pairs, buf.lt, buf.ray_off, None, dl, buf.grad, buf.counts, buf.workspace)
    assert e.value.status == 1
    g.sh_degree = 3
    with pytest.raises(AssertionError):
        g.c()
    assert G.lib().gart_status_string(3) == b"capacity exceeded"
    torch.cuda.synchronize()


def test_host_entry_point_matches_device_path():
    scene, cams = gs.config_cluster(n=2000, width=96, height=64)
    cam, cfg = cams[0], G.Config(tile_size=8, lt_layout=G.LT_PRIMITIVE_MAJOR)
    g = gs.upstream_gradient(cam, 0)
    gpu = P.run_gpu(scene, cam, cfg, g, atomic=False)
    Pn, Hn = gpu["counts"][G.CNT_PAIRS], gpu["counts"][G.CNT_HITS]
    Ln = G.size_view(cfg, gpu["g"], cam)[1]      # a hit capacity that holds either LT layout with its padding

    class HS:
        pass
    hs = HS()
    for k in ("mean", "scale", "quat", "opacity", "sh"):
        setattr(hs, k, torch.from_numpy(getattr(scene, k)).pin_memory())
    hs.sh_degree = scene.sh_degree
    color = torch.empty((cam.height, cam.width, 3), dtype=torch.float32).pin_memory()
    grad = torch.empty((scene.n, G.GRAD_WORDS), dtype=torch.float32).pin_memory()
    arena = torch.empty(G.gart_view_host_arena_bytes(scene.n, scene.sh_degree, cam.width, cam.height, 8, Pn + 5, Ln + 5),
                        dtype=torch.uint8, device="cuda")
    counts = G.gart_view_host(cfg, hs, cam, torch.from_numpy(g).pin_memory(), color, grad, Pn + 5, Ln + 5, arena)
    assert counts[G.CNT_HITS] == Hn and counts[G.CNT_PAIRS] == Pn
    assert np.array_equal(color.numpy(), gpu["color"])
    a, b = grad.numpy().astype(np.float64), gpu["grad"].astype(np.float64)
    assert np.all(np.abs(a - b) <= 1e-4 * np.abs(b) + 1e-5 * np.abs(b).max(axis=1, keepdims=True) + 1e-7)
    with pytest.raises(G.GartError) as e:
        G.gart_view_host(cfg, hs, cam, torch.from_numpy(g).pin_memory(), color, grad, Pn + 5, Hn // 2, arena)
    assert e.value.status == 3
    # the tile-major layout through the host entry point runs the block-per-tile pass: same gradient up to summation order
    G.gart_view_host(G.Config(tile_size=8, lt_layout=G.LT_TILE_MAJOR), hs, cam, torch.from_numpy(g).pin_memory(), color, grad, Pn + 5, Ln + 5, arena)
    assert np.array_equal(color.numpy(), gpu["color"])
    a = grad.numpy().astype(np.float64)
    assert np.all(np.abs(a - b) <= 1e-3 * np.abs(b) + 1e-5 * np.abs(b).max(axis=1, keepdims=True) + 1e-7)
    # the configuration travels through the host entry point: a hit cap with 8-byte LT entries gives the device path's result
    cfg2 = G.Config(tile_size=8, max_hits=4, lt_format=2, lt_layout=G.LT_TILE_MAJOR)
    gpu2 = P.run_gpu(scene, cam, dataclasses.replace(cfg2, lt_format=0, lt_layout=G.LT_PRIMITIVE_MAJOR), g, atomic=True)
    G.gart_view_host(cfg2, hs, cam, torch.from_numpy(g).pin_memory(), color, grad, Pn + 5, Ln + 5, arena)
    assert np.array_equal(color.numpy(), gpu2["color"]) and np.abs(gpu2["color"] - gpu["color"]).max() > 1e-3
    a, b = grad.numpy().astype(np.float64), gpu2["grad_lt16"].astype(np.float64)
    assert np.all(np.abs(a - b) <= 1e-4 * np.abs(b) + 1e-5 * np.abs(b).max(axis=1, keepdims=True) + 1e-7)
    # two views in flight on two streams (gart_view_host_async), each with its own arena and host arrays: the results of
    # the one-at-a-time calls, to the bit for colour and, for the item pass on Gaussians that are one item, for the gradient
    cfg = G.Config(tile_size=8, lt_layout=G.LT_PRIMITIVE_MAJOR)
    want = []
    for v in (0, 1):
        gv = torch.from_numpy(gs.upstream_gradient(cam, v)).pin_memory()
        G.gart_view_host(cfg, hs, cam, gv, color, grad, Pn + 5, Ln + 5, arena)
        want.append((gv, color.clone(), grad.clone()))
    slots = []
    for v in (0, 1):
        slots.append({"color": torch.empty_like(color).pin_memory(), "grad": torch.empty_like(grad).pin_memory(),
                      "counts": torch.zeros(G.COUNTS_WORDS, dtype=torch.int32).pin_memory(), "stream": torch.cuda.Stream(),
                      "arena": torch.empty_like(arena)})
    torch.cuda.synchronize()
    for v, sl in enumerate(slots):
        G.gart_view_host_async(cfg, hs, cam, want[v][0], sl["color"], sl["grad"], Pn + 5, Ln + 5, sl["counts"], sl["arena"], sl["stream"])
    for v, sl in enumerate(slots):
        sl["stream"].synchronize()
        assert G.gart_counts_status(sl["counts"]) == G.GART_OK
        assert sl["counts"].numpy().view(np.uint32)[G.CNT_HITS] == Hn
        assert np.array_equal(sl["color"].numpy(), want[v][1].numpy())
        a, b = sl["grad"].numpy().astype(np.float64), want[v][2].numpy().astype(np.float64)
        assert np.all(np.abs(a - b) <= 1e-4 * np.abs(b) + 1e-5 * np.abs(b).max(axis=1, keepdims=True) + 1e-7)
    assert np.abs(slots[0]["grad"].numpy() - slots[1]["grad"].numpy()).max() > 0      # (two different upstream gradients)
    # a capacity error shows in the counts block once the stream is done
    sl = slots[0]
    G.gart_view_host_async(cfg, hs, cam, want[0][0], sl["color"], sl["grad"], Pn + 5, Hn // 2, sl["counts"], sl["arena"], sl["stream"])
    sl["stream"].synchronize()
    assert G.gart_counts_status(sl["counts"]) == 3
