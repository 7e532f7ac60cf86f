"""Seeded synthetic scenes and cameras for the Gaussian ray-tracing hot path.

This module only draws random inputs (Gaussian parameters, cameras, upstream
gradients).  It contains none of the method's arithmetic: no bounds, no hit
tests, no compositing.  Both the float64 oracle's tests and the CUDA path's
tests / benchmark obtain their inputs from here, so the two sides see the
very same fp32 arrays.

Conventions
-----------
* Camera frame: x right, y down, z forward (the viewing direction).
* ``w2c`` is the 3x4 row-major world-to-camera matrix ``[R | t]``.
* Pinhole intrinsics ``fx, fy, cx, cy`` in pixels; pixel (x, y) has its
  centre at (x + 0.5, y + 0.5).
* Quaternions are (w, x, y, z), unit length before the cast to fp32 and
  used as cast.
* ``sh`` has shape [n, K, 3] with K = (degree + 1)^2, coefficient-major,
  channel-minor.

The five configurations follow the workload list of the benchmark: a tiny
single view, a 10k cluster, an object-centric shell seen from an orbit, and
two unbounded-scene mixtures (dense foreground ball + far background shell)
at the 1237x822 image shape of outdoor captures down-sampled by four.
Draw order per configuration: means, scales, quaternions, opacities, SH
(DC then higher bands), upstream gradient.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np


@dataclasses.dataclass
class Camera:
    width: int
    height: int
    fx: float
    fy: float
    cx: float
    cy: float
    w2c: np.ndarray  # [3, 4] float64, row-major [R | t]

    def as_tuple(self):
        return (self.width, self.height, self.fx, self.fy, self.cx, self.cy,
                np.ascontiguousarray(self.w2c, dtype=np.float64))


@dataclasses.dataclass
class Scene:
    mean: np.ndarray      # [n, 3] float32
    scale: np.ndarray     # [n, 3] float32
    quat: np.ndarray      # [n, 4] float32 (w, x, y, z)
    opacity: np.ndarray   # [n]    float32 in (0, 1)
    sh: np.ndarray        # [n, K, 3] float32
    sh_degree: int

    @property
    def n(self) -> int:
        return int(self.mean.shape[0])

    def subset(self, idx) -> "Scene":
        return Scene(self.mean[idx].copy(), self.scale[idx].copy(), self.quat[idx].copy(),
                     self.opacity[idx].copy(), self.sh[idx].copy(), self.sh_degree)


def pinhole(width: int, height: int, fov_x_deg: float, w2c=None) -> Camera:
    fx = width / (2.0 * math.tan(math.radians(fov_x_deg) / 2.0))
    if w2c is None:
        w2c = np.concatenate([np.eye(3), np.zeros((3, 1))], axis=1)
    return Camera(width, height, fx, fx, width / 2.0, height / 2.0, np.asarray(w2c, dtype=np.float64))


def look_at(position, target=(0.0, 0.0, 0.0), down=(0.0, 1.0, 0.0)) -> np.ndarray:
    """World-to-camera [R | t] for a camera at ``position`` looking at ``target``.

    The world's "down" direction is +y, matching the camera frame's y-down axis.
    """
    p = np.asarray(position, dtype=np.float64)
    f = np.asarray(target, dtype=np.float64) - p
    f /= np.linalg.norm(f)
    r = np.cross(np.asarray(down, dtype=np.float64), f)
    r /= np.linalg.norm(r)
    d = np.cross(f, r)
    R = np.stack([r, d, f], axis=0)
    t = -R @ p
    return np.concatenate([R, t[:, None]], axis=1)


def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def _unit_quats(rng, n):
    q = rng.standard_normal((n, 4))
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    return q


def _sh(rng, n, degree):
    """DC ~ U(0,1), higher bands ~ N(0, 0.1); drawn in fp32 (the arrays are fp32 anyway)."""
    K = (degree + 1) ** 2
    sh = np.empty((n, K, 3), dtype=np.float32)
    sh[:, 0, :] = rng.random((n, 3), dtype=np.float32)
    if K > 1:
        sh[:, 1:, :] = rng.standard_normal((n, K - 1, 3), dtype=np.float32) * np.float32(0.1)
    return sh


def _pack(mean, scale, quat, opacity, sh, degree) -> Scene:
    f32 = lambda a: np.ascontiguousarray(a, dtype=np.float32)
    return Scene(f32(mean), f32(scale), f32(quat), f32(opacity), f32(sh), degree)


def upstream_gradient(cam: Camera, seed: int) -> np.ndarray:
    """dL/dC ~ N(0, 1), shape [height, width, 3], fp32."""
    rng = np.random.default_rng([seed, 0x9D])
    return rng.standard_normal((cam.height, cam.width, 3)).astype(np.float32)


# --------------------------------------------------------------------------
# configurations
# --------------------------------------------------------------------------

def config_tiny(seed: int = 0, n: int = 256, sh_degree: int = 0, width: int = 64, height: int = 64):
    """64x64 view from the origin along +z, fov 50 degrees, 256 Gaussians in a slab."""
    rng = np.random.default_rng(seed)
    mean = np.concatenate([rng.uniform(-1.0, 1.0, (n, 2)), rng.uniform(2.0, 4.0, (n, 1))], axis=1)
    scale = np.exp(rng.uniform(math.log(0.01), math.log(0.1), (n, 3)))
    quat = _unit_quats(rng, n)
    opacity = _sigmoid(rng.normal(0.0, 1.0, n))
    sh = _sh(rng, n, sh_degree)
    cam = pinhole(width, height, 50.0)
    return _pack(mean, scale, quat, opacity, sh, sh_degree), [cam]


def config_cluster(seed: int = 0, n: int = 10_000, sh_degree: int = 3, width: int = 256, height: int = 256):
    """256x256 view of a unit-cube cluster centred at depth 3, fov 30 degrees."""
    rng = np.random.default_rng(seed)
    mean = rng.uniform(-0.5, 0.5, (n, 3)) + np.array([0.0, 0.0, 3.0])
    scale = np.exp(rng.uniform(math.log(0.005), math.log(0.05), (n, 3)))
    quat = _unit_quats(rng, n)
    opacity = _sigmoid(rng.normal(0.0, 1.5, n))
    sh = _sh(rng, n, sh_degree)
    cam = pinhole(width, height, 30.0)
    return _pack(mean, scale, quat, opacity, sh, sh_degree), [cam]


def config_shell(seed: int = 0, n: int = 200_000, sh_degree: int = 3, width: int = 800, height: int = 800,
                 n_views: int = 4):
    """Object-centric: Gaussians on a noisy unit sphere shell, orbit of radius 4, fov 40 degrees."""
    rng = np.random.default_rng(seed)
    u = rng.standard_normal((n, 3))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    mean = u * (1.0 + rng.normal(0.0, 0.05, (n, 1)))
    scale = np.exp(rng.normal(math.log(0.01), 0.5, (n, 3)))
    quat = _unit_quats(rng, n)
    opacity = _sigmoid(rng.normal(0.0, 1.5, n))
    sh = _sh(rng, n, sh_degree)
    cams = []
    elev = math.radians(10.0)
    for v in range(n_views):
        az = 2.0 * math.pi * v / n_views
        pos = (4.0 * math.cos(elev) * math.sin(az), -4.0 * math.sin(elev), -4.0 * math.cos(elev) * math.cos(az))
        cams.append(pinhole(width, height, 40.0, look_at(pos)))
    return _pack(mean, scale, quat, opacity, sh, sh_degree), cams


def _unbounded(rng, n, fg_log_scale, fg_sigma, bg_log_scale, bg_sigma, sh_degree):
    n_fg = int(round(0.7 * n))
    n_bg = n - n_fg
    # foreground: uniform in a ball of radius 2
    u = rng.standard_normal((n_fg, 3))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    mean_fg = u * (2.0 * rng.uniform(0.0, 1.0, (n_fg, 1)) ** (1.0 / 3.0))
    # background: shell, radius uniform in [10, 50]
    w = rng.standard_normal((n_bg, 3))
    w /= np.linalg.norm(w, axis=1, keepdims=True)
    r_bg = rng.uniform(10.0, 50.0, (n_bg, 1))
    mean = np.concatenate([mean_fg, w * r_bg], axis=0)
    s_fg = np.exp(rng.normal(fg_log_scale, fg_sigma, (n_fg, 3)))
    s_bg = np.minimum(2.0, np.exp(rng.normal(bg_log_scale, bg_sigma, (n_bg, 3))) * r_bg / 10.0)
    scale = np.concatenate([s_fg, s_bg], axis=0)
    # interleave foreground and background so that ids carry no depth information
    perm = rng.permutation(n)
    mean, scale = mean[perm], scale[perm]
    quat = _unit_quats(rng, n)
    opacity = _sigmoid(rng.normal(1.0, 1.0, n))
    sh = _sh(rng, n, sh_degree)
    return _pack(mean, scale, quat, opacity, sh, sh_degree)


def unbounded_camera(view: int = 0, n_orbit: int = 64, width: int = 1237, height: int = 822) -> Camera:
    """Camera ``view`` of the elliptical orbit (5 cos phi, -0.8, 4 sin phi), fov_x 60 degrees."""
    phi = 2.0 * math.pi * view / n_orbit
    pos = (5.0 * math.cos(phi), -0.8, 4.0 * math.sin(phi))
    return pinhole(width, height, 60.0, look_at(pos))


def config_unbounded_1m(seed: int = 0, n: int = 1_000_000, sh_degree: int = 3, width: int = 1237,
                        height: int = 822, n_views: int = 1):
    """1M Gaussians: 70% foreground ball (radius 2) + 30% background shell (radius 10..50)."""
    rng = np.random.default_rng(seed)
    scene = _unbounded(rng, n, math.log(0.008), 0.5, math.log(0.03), 0.7, sh_degree)
    return scene, [unbounded_camera(v, 64, width, height) for v in range(n_views)]


def config_unbounded_6m(seed: int = 0, n: int = 6_000_000, sh_degree: int = 3, width: int = 1237,
                        height: int = 822, n_views: int = 16):
    """6M Gaussians, same mixture with smaller primitives, 16 consecutive orbit views."""
    rng = np.random.default_rng(seed)
    scene = _unbounded(rng, n, math.log(0.0045), 0.5, math.log(0.017), 0.7, sh_degree)
    return scene, [unbounded_camera(v, 64, width, height) for v in range(n_views)]


CONFIGS = {
    "tiny": config_tiny,
    "cluster10k": config_cluster,
    "shell200k": config_shell,
    "unbounded1m": config_unbounded_1m,
    "unbounded6m": config_unbounded_6m,
}


def make(name: str, **kw):
    return CONFIGS[name](**kw)
