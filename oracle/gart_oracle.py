"""ctypes binding of the float64 CPU oracle (``gart_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA package never imports this module.

The binding widens fp32 scene arrays to float64 exactly and keeps them alive
for the lifetime of the objects that reference them.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gart_oracle.c")
_LIB = os.path.join(_HERE, "build", "libgart_oracle.so")

ALPHA_MIN = 1.0 / 255.0
NEAR = 0.01


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP) if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Camera(C.Structure):
    _fields_ = [("width", C.c_int32), ("height", C.c_int32), ("fx", C.c_double), ("fy", C.c_double),
                ("cx", C.c_double), ("cy", C.c_double), ("w2c", C.c_double * 12)]


class _Scene(C.Structure):
    _fields_ = [("n", C.c_int64), ("sh_degree", C.c_int32), ("mean", C.c_void_p), ("scale", C.c_void_p),
                ("quat", C.c_void_p), ("opacity", C.c_void_p), ("sh", C.c_void_p)]


class _Config(C.Structure):
    _fields_ = [("alpha_min", C.c_double), ("near_z", C.c_double), ("bg", C.c_double * 3), ("max_hits", C.c_int64),
                ("t_min", C.c_double), ("alpha_max", C.c_double), ("kernel_degree", C.c_int64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_max_threads.restype = C.c_int
        L.orc_set_threads.argtypes = [C.c_int]
        L.orc_sh_basis.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_ray.argtypes = [C.POINTER(_Camera), C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_bounds.argtypes = [C.POINTER(_Scene), C.POINTER(_Camera), C.POINTER(_Config), C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_tile_map.argtypes = [C.c_int64, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.POINTER(C.c_int64)]
        L.orc_tile_map.restype = C.c_int64
        L.orc_view_create.argtypes = [C.POINTER(_Scene), C.POINTER(_Camera), C.POINTER(_Config)]
        L.orc_view_create.restype = C.c_void_p
        L.orc_view_destroy.argtypes = [C.c_void_p]
        L.orc_view_eval_pair.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p]
        L.orc_view_find_hits.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        L.orc_view_find_hits.restype = C.c_int64
        L.orc_view_set_hits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_view_num_hits.argtypes = [C.c_void_p]
        L.orc_view_num_hits.restype = C.c_int64
        L.orc_view_get_hits.argtypes = [C.c_void_p] + [C.c_void_p] * 4
        L.orc_view_composite.argtypes = [C.c_void_p] + [C.c_void_p] * 3
        L.orc_view_backward.argtypes = [C.c_void_p] + [C.c_void_p] * 6
        L.orc_view_backward.restype = C.c_int
        L.orc_view_lt_entries.argtypes = [C.c_void_p] + [C.c_void_p] * 3
        L.orc_view_lt_entries.restype = C.c_int
        L.orc_view_margins.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_view_ray_margins.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_view_ray_margins.restype = C.c_int
        _lib = L
    return _lib


def max_threads() -> int:
    return lib().orc_max_threads()


def set_threads(t: int) -> None:
    lib().orc_set_threads(int(t))


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _camera(cam) -> _Camera:
    c = _Camera()
    c.width, c.height = int(cam.width), int(cam.height)
    c.fx, c.fy, c.cx, c.cy = float(cam.fx), float(cam.fy), float(cam.cx), float(cam.cy)
    w = _f64(cam.w2c).reshape(12)
    for i in range(12):
        c.w2c[i] = w[i]
    return c


def _config(alpha_min, near, bg, max_hits=0, t_min=0.0, alpha_max=1.0, kernel_degree=2) -> _Config:
    c = _Config()
    c.kernel_degree = int(kernel_degree)
    c.alpha_min, c.near_z = float(alpha_min), float(near)
    c.max_hits = int(max_hits)
    c.t_min, c.alpha_max = float(t_min), float(alpha_max)
    for i in range(3):
        c.bg[i] = float(bg[i])
    return c


class OracleScene:
    """Scene arrays widened to float64; accepts fp32 or fp64 inputs."""

    def __init__(self, mean, scale, quat, opacity, sh, sh_degree):
        self.mean, self.scale, self.quat = _f64(mean), _f64(scale), _f64(quat)
        self.opacity, self.sh = _f64(opacity), _f64(sh)
        self.sh_degree = int(sh_degree)
        self.n = int(self.mean.shape[0])
        self.K = (self.sh_degree + 1) ** 2
        assert self.sh.shape == (self.n, self.K, 3), self.sh.shape
        s = _Scene()
        s.n, s.sh_degree = self.n, self.sh_degree
        s.mean, s.scale, s.quat = _ptr(self.mean), _ptr(self.scale), _ptr(self.quat)
        s.opacity, s.sh = _ptr(self.opacity), _ptr(self.sh)
        self.c = s

    @classmethod
    def from_scene(cls, sc):
        return cls(sc.mean, sc.scale, sc.quat, sc.opacity, sc.sh, sc.sh_degree)

    @property
    def grad_words(self):
        return 11 + 3 * self.K


def sh_basis(d) -> np.ndarray:
    d = _f64(d)
    out = np.zeros(16)
    lib().orc_sh_basis(_ptr(d), _ptr(out))
    return out


def ray(cam, x, y):
    o, d = np.zeros(3), np.zeros(3)
    c = _camera(cam)
    lib().orc_ray(C.byref(c), int(x), int(y), _ptr(o), _ptr(d))
    return o, d


def bounds(scene: OracleScene, cam, alpha_min=ALPHA_MIN, near=NEAR, kernel_degree=2):
    """Eq. 9-14: returns rect [n,4] int32 (x0,y0,x1,y1 inclusive), cls [n] uint8, margin [n] float64.
    kernel_degree k: the response is exp(-D^k / 2) (k = 2: Eq. 4), so the clamping radius is (2 ln(sigma/alpha_min))^(1/k)."""
    rect = np.zeros((scene.n, 4), dtype=np.int32)
    cls = np.zeros(scene.n, dtype=np.uint8)
    margin = np.zeros(scene.n, dtype=np.float64)
    c, g = _camera(cam), _config(alpha_min, near, (0, 0, 0), kernel_degree=kernel_degree)
    lib().orc_bounds(C.byref(scene.c), C.byref(c), C.byref(g), _ptr(rect), _ptr(cls), _ptr(margin))
    return rect, cls, margin


def tile_map(rect, width, height, ts):
    """Tile lists: returns tile_off [T+1] uint32, pair_gid [P] uint32, slots (sum of rectangle areas)."""
    rect = np.ascontiguousarray(rect, dtype=np.int32)
    n = rect.shape[0]
    T = ((width + ts - 1) // ts) * ((height + ts - 1) // ts)
    tile_off = np.zeros(T + 1, dtype=np.uint32)
    slots = C.c_int64(0)
    P = lib().orc_tile_map(n, _ptr(rect), width, height, ts, _ptr(tile_off), None, C.byref(slots))
    pair_gid = np.zeros(max(P, 1), dtype=np.uint32)
    lib().orc_tile_map(n, _ptr(rect), width, height, ts, _ptr(tile_off), _ptr(pair_gid), C.byref(slots))
    return tile_off, pair_gid[:P], int(slots.value)


BRUTE = 0      # every requested ray against every Gaussian not culled by rule
PREFILTER = 1  # candidates from the projected bounding sphere, padded by one pixel


class View:
    """One camera view of a scene: hit discovery, ordering, compositing, backward."""

    def __init__(self, scene: OracleScene, cam, alpha_min=ALPHA_MIN, near=NEAR, bg=(0.0, 0.0, 0.0), max_hits=0, t_min=0.0,
                 alpha_max=1.0, kernel_degree=2):
        """max_hits > 0 composites only the first max_hits hits of every ray (0: all of them); t_min > 0 ends a ray before
        the first hit with less than t_min transmittance in front of it; alpha_max < 1 clamps every hit's alpha;
        kernel_degree k > 2 (even) makes the response exp(-D^k / 2), a narrow kernel (k = 2: the Gaussian of Eq. 4)."""
        self.scene, self.cam = scene, cam
        self._c, self._g = _camera(cam), _config(alpha_min, near, bg, max_hits, t_min, alpha_max, kernel_degree)
        self.n_rays = int(cam.width) * int(cam.height)
        self._h = lib().orc_view_create(C.byref(scene.c), C.byref(self._c), C.byref(self._g))
        self._keep = None

    def close(self):
        if self._h:
            lib().orc_view_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def eval_pair(self, ray_index, gid):
        """(alpha, t*) of one ray-Gaussian pair, no threshold applied."""
        out = np.zeros(2)
        lib().orc_view_eval_pair(self._h, int(ray_index), int(gid), _ptr(out))
        return float(out[0]), float(out[1])

    def find_hits(self, mode=BRUTE, pixel_mask=None) -> int:
        if pixel_mask is not None:
            pixel_mask = np.ascontiguousarray(pixel_mask, dtype=np.uint8).reshape(-1)
            assert pixel_mask.size == self.n_rays
        return int(lib().orc_view_find_hits(self._h, int(mode), _ptr(pixel_mask)))

    def set_hits(self, ray_off, ray_gid):
        ray_off = np.ascontiguousarray(ray_off, dtype=np.uint64)
        ray_gid = np.ascontiguousarray(ray_gid, dtype=np.uint32)
        assert ray_off.size == self.n_rays + 1 and int(ray_off[-1]) <= ray_gid.size
        lib().orc_view_set_hits(self._h, _ptr(ray_off), _ptr(ray_gid))

    def hits(self):
        """(ray_off [n_rays+1] uint64, gid [H] uint32, t* [H], alpha [H])."""
        H = int(lib().orc_view_num_hits(self._h))
        ray_off = np.zeros(self.n_rays + 1, dtype=np.uint64)
        gid = np.zeros(max(H, 1), dtype=np.uint32)
        t = np.zeros(max(H, 1))
        a = np.zeros(max(H, 1))
        lib().orc_view_get_hits(self._h, _ptr(ray_off), _ptr(gid), _ptr(t), _ptr(a))
        return ray_off, gid[:H], t[:H], a[:H]

    def composite(self):
        """Eq. 6-8: (color [H,W,3], t_final [H,W], hit_count [H,W] uint32)."""
        h, w = self.cam.height, self.cam.width
        color = np.zeros((h, w, 3))
        t_final = np.zeros((h, w))
        cnt = np.zeros((h, w), dtype=np.uint32)
        lib().orc_view_composite(self._h, _ptr(color), _ptr(t_final), _ptr(cnt))
        return color, t_final, cnt

    def margins(self):
        """(min |ln(T_i / t_min)| over the termination tests, min |ln(alpha / alpha_max)| over the composited hits) of
        the last composite(): how close a floating-point decision of the two options came to flipping."""
        out = np.zeros(2)
        lib().orc_view_margins(self._h, _ptr(out))
        return float(out[0]), float(out[1])

    def ray_margins(self):
        """The same two margins per ray, [n_rays, 2] (infinity where a ray met no such decision)."""
        out = np.zeros((self.n_rays, 2))
        if lib().orc_view_ray_margins(self._h, _ptr(out)) != 0:
            raise RuntimeError("composite() must run before ray_margins()")
        return out

    def backward(self, dL_dC, with_abs=False, with_elem=False, with_terms=False, with_cond=False):
        """Gradients [n, 11+3K] (mean 3, scale 3, quat 4, opacity 1, sh K*3) of sum <dL_dC, C>.
        with_abs adds the sums of absolute per-hit contributions, with_elem those of the contributions
        split by colour channel (the scale of an error that is relative to the per-hit quantities), with_terms
        those with each channel's term split again into its two products (hit colour against colour behind), with_cond
        the first-order effect, per unit of relative error of every alpha, on each word through the transmittances."""
        g = _f64(dL_dC).reshape(self.n_rays, 3)
        G = self.scene.grad_words
        grad = np.zeros((self.scene.n, G))
        gabs = np.zeros((self.scene.n, G)) if with_abs else None
        gelem = np.zeros((self.scene.n, G)) if with_elem else None
        gterms = np.zeros((self.scene.n, G)) if with_terms else None
        gcond = np.zeros((self.scene.n, G)) if with_cond else None
        rc = lib().orc_view_backward(self._h, _ptr(g), _ptr(grad), _ptr(gabs), _ptr(gelem), _ptr(gterms), _ptr(gcond))
        if rc != 0:
            raise RuntimeError("composite() must run before backward()")
        out = ((grad,) + ((gabs,) if with_abs else ()) + ((gelem,) if with_elem else ()) + ((gterms,) if with_terms else ())
               + ((gcond,) if with_cond else ()))
        return out if len(out) > 1 else grad

    def lt_entries(self, with_cond=False):
        """Per hit, in list order: (entry [H,4] = alpha dC/dalpha (3) and w = T alpha; flags [H] uint8, bit ch set
        where colour channel ch is not clamped); with_cond adds cond [H,4], the first-order effect on each word of a
        unit relative error of every alpha on the ray."""
        H = int(lib().orc_view_num_hits(self._h))
        entry = np.zeros((max(H, 1), 4))
        flags = np.zeros(max(H, 1), dtype=np.uint8)
        cond = np.zeros((max(H, 1), 4)) if with_cond else None
        if lib().orc_view_lt_entries(self._h, _ptr(entry), _ptr(flags), _ptr(cond)) != 0:
            raise RuntimeError("composite() must run before lt_entries()")
        return (entry[:H], flags[:H], cond[:H]) if with_cond else (entry[:H], flags[:H])


def render(scene: OracleScene, cam, dL_dC=None, mode=BRUTE, pixel_mask=None, hit_lists=None, **kw):
    """Convenience: discover (or impose) hits, composite and optionally run the backward."""
    v = View(scene, cam, **kw)
    if hit_lists is not None:
        v.set_hits(*hit_lists)
    else:
        v.find_hits(mode, pixel_mask)
    color, t_final, cnt = v.composite()
    out = {"view": v, "color": color, "t_final": t_final, "hit_count": cnt}
    if dL_dC is not None:
        out["grad"] = v.backward(dL_dC)
    return out
