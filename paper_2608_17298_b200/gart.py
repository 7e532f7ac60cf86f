"""Thin Python binding of ``libgart.so`` (ctypes).

Only argument marshalling lives here: PyTorch provides device memory and streams, every step
of the path runs in the CUDA library.  The functions carry the names of the C entry points
(``include/gart.h``) and take torch CUDA tensors where the C ABI takes device pointers.

The library must have been built (``python -m paper_2608_17298_b200.build``); loading fails
loudly otherwise -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgart.so")

GART_OK = 0
STATUS_NAMES = {0: "GART_OK", 1: "GART_ERR_INVALID_ARG", 2: "GART_ERR_WORKSPACE_TOO_SMALL",
                3: "GART_ERR_CAPACITY_EXCEEDED", 4: "GART_ERR_CUDA", 5: "GART_ERR_TIMEOUT"}
LT_PRIMITIVE_MAJOR, LT_TILE_MAJOR = 0, 1
# names of the arrays inside the view block (gart_view_array): index, numpy-style dtype width in bytes, columns
VIEW_ARRAYS = {"pair_mask": 0, "pair_order": 1, "rank_sid": 2, "rank_mask": 3, "rank_gstart": 4, "tile_lt_base": 5,
               "pair_gpos": 6, "gpair_off": 7, "gm_mask": 8, "gm_ltb": 9, "item_desc": 10, "item_gstart": 11,
               "st_off": 12, "st_lt_base": 13, "info": 14}
CNT_VISIBLE, CNT_PAIRS, CNT_SLOTS_LO, CNT_SLOTS_HI, CNT_HITS, CNT_ERROR, CNT_MAX_RAY_HITS, CNT_STRADDLE, CNT_LT_SLOTS = range(9)
COUNTS_WORDS = 12
GRAD_WORDS = 64

EXPORTS = [
    "gart_status_string", "gart_mask_words", "gart_pre_words", "gart_bounds_workspace_bytes", "gart_bounds",
    "gart_tile_map_workspace_bytes", "gart_tile_map", "gart_tile_map_static", "gart_view_bytes", "gart_view_array",
    "gart_forward_workspace_bytes", "gart_forward",
    "gart_backward_workspace_bytes", "gart_backward_hybrid_workspace_bytes", "gart_backward", "gart_backward_tile", "gart_backward_atomic", "gart_backward_hybrid",
    "gart_backward_warp",
    "gart_workspace_bytes", "gart_read_counts", "gart_sync_status",
    "gart_view_host_arena_bytes", "gart_view_host", "gart_view_host_async", "gart_counts_status",
]


class GartError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s returned %s" % (where, STATUS_NAMES.get(int(status), status)))


class _Config(C.Structure):
    _fields_ = [("alpha_min", C.c_float), ("near_z", C.c_float), ("background", C.c_float * 3), ("tile_size", C.c_int32),
                ("lt_format", C.c_int32), ("max_hits", C.c_int32), ("lt_layout", C.c_int32), ("t_min", C.c_float),
                ("alpha_max", C.c_float), ("atomic_mode", C.c_int32), ("wait_polls", C.c_int32), ("kernel_degree", C.c_int32)]


class _Camera(C.Structure):
    _fields_ = [("width", C.c_int32), ("height", C.c_int32), ("fx", C.c_double), ("fy", C.c_double),
                ("cx", C.c_double), ("cy", C.c_double), ("w2c", C.c_double * 12)]


class _Gaussians(C.Structure):
    _fields_ = [("n", C.c_int64), ("sh_degree", C.c_int32), ("mean", C.c_void_p), ("scale", C.c_void_p),
                ("quat", C.c_void_p), ("opacity", C.c_void_p), ("sh", C.c_void_p)]


_lib = None


def lib():
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libgart.so is missing: build it with `python -m paper_2608_17298_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        L.gart_status_string.restype = C.c_char_p
        L.gart_status_string.argtypes = [C.c_int]
        L.gart_mask_words.restype = i32
        L.gart_mask_words.argtypes = [i32]
        L.gart_pre_words.restype = i32
        L.gart_pre_words.argtypes = [i32]
        L.gart_bounds_workspace_bytes.restype = sz
        L.gart_bounds_workspace_bytes.argtypes = [i64]
        L.gart_bounds.argtypes = [vp] * 10 + [sz, vp]
        L.gart_tile_map_workspace_bytes.restype = sz
        L.gart_tile_map_workspace_bytes.argtypes = [i64, i32, i32, i32, i64]
        L.gart_tile_map.argtypes = [vp, vp, i64, i32, i32, vp, vp, i64, vp, vp, sz, vp]
        L.gart_tile_map_static.argtypes = [vp, vp, i64, i32, i32, vp, vp, i64, vp, vp]
        L.gart_tile_map_static.restype = C.c_int
        L.gart_forward_workspace_bytes.restype = sz
        L.gart_forward_workspace_bytes.argtypes = [i32, i32, i32, i64, i64]
        L.gart_view_bytes.restype = sz
        L.gart_view_bytes.argtypes = [i64, i32, i32, i32, i64]
        L.gart_view_array.argtypes = [i64, i32, i32, i32, i64, i32, C.POINTER(sz), C.POINTER(sz)]
        L.gart_forward.argtypes = [vp] * 8 + [i64] + [vp] * 4 + [i64] + [vp] * 4 + [sz, vp, vp, sz, vp]
        L.gart_backward_workspace_bytes.restype = sz
        L.gart_backward_workspace_bytes.argtypes = [i64]
        L.gart_backward_hybrid_workspace_bytes.restype = sz
        L.gart_backward_hybrid_workspace_bytes.argtypes = [i64, i32]
        for fn in ("gart_backward", "gart_backward_tile", "gart_backward_warp"):
            getattr(L, fn).argtypes = [vp] * 8 + [sz, i64] + [vp] * 5 + [sz, vp]
        L.gart_backward_atomic.argtypes = [vp] * 13
        L.gart_backward_hybrid.argtypes = [vp] * 8 + [sz, i64] + [vp] * 7 + [sz, vp]
        L.gart_workspace_bytes.restype = sz
        L.gart_workspace_bytes.argtypes = [i64, i32, i32, i32, i64, i64]
        L.gart_read_counts.argtypes = [vp, vp, vp]
        L.gart_sync_status.argtypes = [vp, vp, vp]
        L.gart_view_host_arena_bytes.restype = sz
        L.gart_view_host_arena_bytes.argtypes = [i64, i32, i32, i32, i32, i64, i64]
        L.gart_view_host.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, vp, vp, sz, vp]
        L.gart_view_host_async.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, vp, vp, sz, vp]
        L.gart_counts_status.argtypes = [vp]
        for fn in ("gart_bounds", "gart_tile_map", "gart_forward", "gart_backward", "gart_backward_tile", "gart_backward_atomic",
                   "gart_backward_hybrid", "gart_backward_warp", "gart_read_counts", "gart_sync_status", "gart_view_host", "gart_view_host_async", "gart_counts_status", "gart_view_array"):
            getattr(L, fn).restype = C.c_int
        _lib = L
    return _lib


# ----------------------------------------------------------------------------------------- host structs
@dataclasses.dataclass
class Config:
    alpha_min: float = 1.0 / 255.0
    near_z: float = 0.01
    background: tuple = (0.0, 0.0, 0.0)
    tile_size: int = 8
    lt_format: int = 0          # 0: 16-byte LT entries (gart_backward); 1: 4 bytes per hit (gart_backward_hybrid); 2: 8 bytes (gart_backward)
    max_hits: int = 0           # > 0: only the first max_hits hits of a ray are composited (0: all, the paper's setting)
    lt_layout: int = LT_TILE_MAJOR   # LT_TILE_MAJOR (1, the faster whole step: block-per-tile backward) or LT_PRIMITIVE_MAJOR (0: item backward, half the DRAM traffic)
    t_min: float = 0.0          # > 0: a ray ends before the first hit with less than t_min transmittance in front (0: off)
    alpha_max: float = 1.0      # < 1: every hit's alpha is clamped to alpha_max (>= 1: off)
    atomic_mode: int = 0        # gart_backward_atomic: 0 scalar atomicAdd per word, 1 one 16-byte vector reduction per four words
    wait_polls: int = 0         # 0: library limit on a kernel's waits for its own copies; > 0: polls; < 0: every wait gives up (test hook)
    kernel_degree: int = 2      # k of the response exp(-D^k / 2): 2 the Gaussian (the paper's setting), 4 a narrow kernel

    def c(self) -> _Config:
        s = _Config()
        s.alpha_min, s.near_z, s.tile_size = self.alpha_min, self.near_z, int(self.tile_size)
        s.lt_format = int(self.lt_format)
        s.max_hits = int(self.max_hits)
        s.lt_layout = int(self.lt_layout)
        s.t_min, s.alpha_max = float(self.t_min), float(self.alpha_max)
        s.wait_polls, s.atomic_mode = int(self.wait_polls), int(self.atomic_mode)
        s.kernel_degree = int(self.kernel_degree)
        for i in range(3):
            s.background[i] = float(self.background[i])
        return s

    @property
    def alpha_min_f32(self) -> float:
        """The threshold as the library sees it (rounded to fp32)."""
        return float(C.c_float(self.alpha_min).value)

    @property
    def near_f32(self) -> float:
        return float(C.c_float(self.near_z).value)

    @property
    def t_min_f32(self) -> float:
        return float(C.c_float(self.t_min).value)

    @property
    def alpha_max_f32(self) -> float:
        return float(C.c_float(self.alpha_max).value)


def camera_struct(cam) -> _Camera:
    """``cam`` has width, height, fx, fy, cx, cy and a [3,4] world-to-camera matrix ``w2c``."""
    s = _Camera()
    s.width, s.height = int(cam.width), int(cam.height)
    s.fx, s.fy, s.cx, s.cy = float(cam.fx), float(cam.fy), float(cam.cx), float(cam.cy)
    flat = [float(v) for row in cam.w2c for v in row]
    for i in range(12):
        s.w2c[i] = flat[i]
    return s


def _dev(t, dtype, what):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return t.data_ptr()


@dataclasses.dataclass
class Gaussians:
    """Device-resident scene: fp32 CUDA tensors mean [n,3], scale [n,3], quat [n,4], opacity [n], sh [n,K,3]."""
    mean: torch.Tensor
    scale: torch.Tensor
    quat: torch.Tensor
    opacity: torch.Tensor
    sh: torch.Tensor
    sh_degree: int

    @property
    def n(self):
        return int(self.mean.shape[0])

    @classmethod
    def from_numpy(cls, scene, device="cuda"):
        f = lambda a: torch.from_numpy(a).to(device=device, dtype=torch.float32).contiguous()
        return cls(f(scene.mean), f(scene.scale), f(scene.quat), f(scene.opacity), f(scene.sh), int(scene.sh_degree))

    def c(self) -> _Gaussians:
        K = (self.sh_degree + 1) ** 2
        n = self.n
        assert self.sh.shape == (n, K, 3) and self.scale.shape == (n, 3) and self.quat.shape == (n, 4)
        s = _Gaussians()
        s.n, s.sh_degree = n, int(self.sh_degree)
        s.mean, s.scale = _dev(self.mean, torch.float32, "mean"), _dev(self.scale, torch.float32, "scale")
        s.quat, s.opacity = _dev(self.quat, torch.float32, "quat"), _dev(self.opacity, torch.float32, "opacity")
        s.sh = _dev(self.sh, torch.float32, "sh")
        return s


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(status, where):
    if status != GART_OK:
        raise GartError(status, where)


def tiles(cam, tile_size):
    return -(-int(cam.width) // tile_size) * -(-int(cam.height) // tile_size)


def gart_mask_words(tile_size: int) -> int:
    return int(lib().gart_mask_words(int(tile_size)))


# ----------------------------------------------------------------------------------------- the calls
def _ws(workspace):
    return _dev(workspace, torch.uint8, "workspace"), (workspace.numel() if workspace is not None else 0)


def gart_pre_words(sh_degree: int) -> int:
    return int(lib().gart_pre_words(int(sh_degree)))


def gart_bounds_workspace_bytes(n) -> int:
    return int(lib().gart_bounds_workspace_bytes(int(n)))


def gart_bounds(cfg: Config, g: Gaussians, cam, rect, cls, pre, slot_of_gid, gid_of_slot, counts, workspace, stream=None):
    c, gs, cs = cfg.c(), g.c(), camera_struct(cam)
    i32 = torch.int32
    wp, wb = _ws(workspace)
    _check(lib().gart_bounds(C.byref(c), C.byref(gs), C.byref(cs), _dev(rect, i32, "rect"), _dev(cls, torch.uint8, "cls"),
                             _dev(pre, torch.float32, "pre"), _dev(slot_of_gid, i32, "slot_of_gid"),
                             _dev(gid_of_slot, i32, "gid_of_slot"), _dev(counts, i32, "counts"), wp, wb,
                             _stream_ptr(stream)), "gart_bounds")


def gart_tile_map_workspace_bytes(n, width, height, tile_size, cap_pairs) -> int:
    return int(lib().gart_tile_map_workspace_bytes(int(n), int(width), int(height), int(tile_size), int(cap_pairs)))


def gart_tile_map(cfg: Config, rect, n, cam, tile_off, pair_gid, cap_pairs, counts, workspace, stream=None):
    c = cfg.c()
    wp, wb = _ws(workspace)
    _check(lib().gart_tile_map(C.byref(c), _dev(rect, torch.int32, "rect"), int(n), int(cam.width), int(cam.height),
                               _dev(tile_off, torch.int32, "tile_off"), _dev(pair_gid, torch.int32, "pair_gid"),
                               int(cap_pairs), _dev(counts, torch.int32, "counts"), wp, wb, _stream_ptr(stream)), "gart_tile_map")


TILE_MAP_STATIC_BYTES = 8 << 20


def gart_tile_map_static(cfg: Config, rect, n, cam, tile_off, pair_gid, cap_pairs, counts, stream=None):
    """gart_tile_map without a workspace argument: the scratch is a fixed array inside the library
    (for callers that cannot allocate device memory when they call).  Problems whose scratch need
    exceeds TILE_MAP_STATIC_BYTES are refused with GART_ERR_WORKSPACE_TOO_SMALL."""
    c = cfg.c()
    _check(lib().gart_tile_map_static(C.byref(c), _dev(rect, torch.int32, "rect"), int(n), int(cam.width), int(cam.height),
                                      _dev(tile_off, torch.int32, "tile_off"), _dev(pair_gid, torch.int32, "pair_gid"),
                                      int(cap_pairs), _dev(counts, torch.int32, "counts"), _stream_ptr(stream)),
           "gart_tile_map_static")


def gart_forward_workspace_bytes(width, height, tile_size, cap_pairs, cap_hits) -> int:
    return int(lib().gart_forward_workspace_bytes(int(width), int(height), int(tile_size), int(cap_pairs), int(cap_hits)))


def gart_workspace_bytes(n, width, height, tile_size, cap_pairs, cap_hits) -> int:
    return int(lib().gart_workspace_bytes(int(n), int(width), int(height), int(tile_size), int(cap_pairs), int(cap_hits)))


def gart_view_bytes(n, width, height, tile_size, cap_pairs) -> int:
    return int(lib().gart_view_bytes(int(n), int(width), int(height), int(tile_size), int(cap_pairs)))


def gart_view_array(n, width, height, tile_size, cap_pairs, name):
    """(offset, bytes) of one named private array inside the view block (tests and diagnostics)."""
    off, nb = C.c_size_t(0), C.c_size_t(0)
    _check(lib().gart_view_array(int(n), int(width), int(height), int(tile_size), int(cap_pairs), VIEW_ARRAYS[name],
                                 C.byref(off), C.byref(nb)), "gart_view_array")
    return int(off.value), int(nb.value)


def _view(view):
    return _dev(view, torch.uint8, "view"), (view.numel() if view is not None else 0)


def gart_forward(cfg: Config, g: Gaussians, cam, pre, slot_of_gid, gid_of_slot, tile_off, pair_gid, cap_pairs, color,
                 t_final, hit_count, lt, cap_hits, ray_off, ray_gid, ray_slot, view, counts, workspace, stream=None):
    c, gs, cs = cfg.c(), g.c(), camera_struct(cam)
    i32, f32 = torch.int32, torch.float32
    wp, wb = _ws(workspace)
    vp, vb = _view(view)
    _check(lib().gart_forward(C.byref(c), C.byref(gs), C.byref(cs), _dev(pre, f32, "pre"),
                              _dev(slot_of_gid, i32, "slot_of_gid"), _dev(gid_of_slot, i32, "gid_of_slot"),
                              _dev(tile_off, i32, "tile_off"), _dev(pair_gid, i32, "pair_gid"), int(cap_pairs),
                              _dev(color, f32, "color"), _dev(t_final, f32, "t_final"), _dev(hit_count, i32, "hit_count"),
                              _dev(lt, f32, "lt"), int(cap_hits), _dev(ray_off, i32, "ray_off"),
                              _dev(ray_gid, i32, "ray_gid"), _dev(ray_slot, i32, "ray_slot"), vp, vb,
                              _dev(counts, i32, "counts"), wp, wb, _stream_ptr(stream)), "gart_forward")


def gart_backward_workspace_bytes(n) -> int:
    return int(lib().gart_backward_workspace_bytes(int(n)))


def gart_backward_hybrid_workspace_bytes(n, sh_degree) -> int:
    return int(lib().gart_backward_hybrid_workspace_bytes(int(n), int(sh_degree)))


def _backward_call(name, cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor, grad, counts,
                   workspace, stream):
    c, gs, cs = cfg.c(), g.c(), camera_struct(cam)
    i32, f32 = torch.int32, torch.float32
    wp, wb = _ws(workspace)
    vp, vb = _view(view)
    _check(getattr(lib(), name)(C.byref(c), C.byref(gs), C.byref(cs), _dev(pre, f32, "pre"),
                                _dev(slot_of_gid, i32, "slot_of_gid"), _dev(gid_of_slot, i32, "gid_of_slot"),
                                _dev(tile_off, i32, "tile_off"), vp, vb, int(cap_pairs),
                                _dev(lt, f32, "lt"), _dev(dL_dcolor, f32, "dL_dcolor"), _dev(grad, f32, "grad"),
                                _dev(counts, i32, "counts"), wp, wb, _stream_ptr(stream)), name)


def gart_backward(cfg: Config, g: Gaussians, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor,
                  grad, counts, workspace, stream=None):
    _backward_call("gart_backward", cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor, grad,
                   counts, workspace, stream)


def gart_backward_tile(cfg: Config, g: Gaussians, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor,
                       grad, counts, workspace, stream=None):
    _backward_call("gart_backward_tile", cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor,
                   grad, counts, workspace, stream)


def gart_backward_warp(cfg: Config, g: Gaussians, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor,
                       grad, counts, workspace, stream=None):
    _backward_call("gart_backward_warp", cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt, dL_dcolor,
                   grad, counts, workspace, stream)


def gart_backward_atomic(cfg: Config, g: Gaussians, cam, pre, slot_of_gid, ray_off, ray_gid, ray_slot, lt, dL_dcolor,
                         grad, counts, stream=None):
    c, gs, cs = cfg.c(), g.c(), camera_struct(cam)
    i32, f32 = torch.int32, torch.float32
    _check(lib().gart_backward_atomic(C.byref(c), C.byref(gs), C.byref(cs), _dev(pre, f32, "pre"),
                                      _dev(slot_of_gid, i32, "slot_of_gid"), _dev(ray_off, i32, "ray_off"),
                                      _dev(ray_gid, i32, "ray_gid"), _dev(ray_slot, i32, "ray_slot"), _dev(lt, f32, "lt"),
                                      _dev(dL_dcolor, f32, "dL_dcolor"), _dev(grad, f32, "grad"),
                                      _dev(counts, i32, "counts"), _stream_ptr(stream)), "gart_backward_atomic")


def gart_backward_hybrid(cfg: Config, g: Gaussians, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, cap_pairs, lt_w, ray_off,
                         ray_gid, dL_dcolor, grad, counts, workspace, stream=None):
    c, gs, cs = cfg.c(), g.c(), camera_struct(cam)
    i32, f32 = torch.int32, torch.float32
    wp, wb = _ws(workspace)
    vp, vb = _view(view)
    _check(lib().gart_backward_hybrid(C.byref(c), C.byref(gs), C.byref(cs), _dev(pre, f32, "pre"),
                                      _dev(slot_of_gid, i32, "slot_of_gid"), _dev(gid_of_slot, i32, "gid_of_slot"),
                                      _dev(tile_off, i32, "tile_off"), vp, vb, int(cap_pairs),
                                      _dev(lt_w, f32, "lt_w"), _dev(ray_off, i32, "ray_off"), _dev(ray_gid, i32, "ray_gid"),
                                      _dev(dL_dcolor, f32, "dL_dcolor"), _dev(grad, f32, "grad"),
                                      _dev(counts, i32, "counts"), wp, wb, _stream_ptr(stream)), "gart_backward_hybrid")


def gart_read_counts(counts, stream=None):
    """Counts block as a list of unsigned ints (synchronises the stream)."""
    host = (C.c_uint32 * COUNTS_WORDS)()
    _check(lib().gart_read_counts(_dev(counts, torch.int32, "counts"), host, _stream_ptr(stream)), "gart_read_counts")
    return [int(v) for v in host]


def gart_sync_status(counts, stream=None) -> int:
    """Reads the counts block (synchronises the stream) and returns its error word as a status code."""
    return int(lib().gart_sync_status(_dev(counts, torch.int32, "counts"), None, _stream_ptr(stream)))


def gart_view_host_arena_bytes(n, sh_degree, width, height, tile_size, cap_pairs, cap_hits) -> int:
    return int(lib().gart_view_host_arena_bytes(int(n), int(sh_degree), int(width), int(height), int(tile_size),
                                                int(cap_pairs), int(cap_hits)))


def _host_ptr(t, what, dtype=torch.float32):
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CPU %s tensor" % (what, dtype))
    return t.data_ptr()


def _host_scene(scene) -> _Gaussians:
    gs = _Gaussians()
    gs.n, gs.sh_degree = int(scene.mean.shape[0]), int(scene.sh_degree)
    gs.mean, gs.scale, gs.quat = _host_ptr(scene.mean, "mean"), _host_ptr(scene.scale, "scale"), _host_ptr(scene.quat, "quat")
    gs.opacity, gs.sh = _host_ptr(scene.opacity, "opacity"), _host_ptr(scene.sh, "sh")
    return gs


def gart_view_host_async(cfg: Config, scene, cam, dL_dcolor, color_out, grad_out, cap_pairs, cap_hits, counts_out, arena, stream=None):
    """gart_view_host without waiting: everything is queued on ``stream``.  ``counts_out`` is a pinned CPU int32 tensor of
    COUNTS_WORDS words; after synchronising the stream, gart_counts_status(counts_out) gives the status."""
    gs = _host_scene(scene)
    c, cs = cfg.c(), camera_struct(cam)
    if counts_out.numel() < COUNTS_WORDS:
        raise ValueError("counts_out must hold COUNTS_WORDS words")
    _check(lib().gart_view_host_async(C.byref(c), C.byref(gs), C.byref(cs), _host_ptr(dL_dcolor, "dL_dcolor"), _host_ptr(color_out, "color_out"),
                                      _host_ptr(grad_out, "grad_out"), int(cap_pairs), int(cap_hits), _host_ptr(counts_out, "counts_out", torch.int32),
                                      _dev(arena, torch.uint8, "arena"), arena.numel(), _stream_ptr(stream)), "gart_view_host_async")


def gart_counts_status(counts_out) -> int:
    return int(lib().gart_counts_status(_host_ptr(counts_out, "counts_out", torch.int32)))


def gart_view_host(cfg: Config, scene, cam, dL_dcolor, color_out, grad_out, cap_pairs, cap_hits, arena, stream=None):
    """End-to-end call on HOST (CPU, ideally pinned) fp32 tensors; ``arena`` is a CUDA uint8 tensor.

    ``scene`` has CPU tensors mean, scale, quat, opacity, sh and ``sh_degree``.  Returns the counts block.
    """
    def host(t, what):
        if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            raise TypeError("%s must be a contiguous CPU float32 tensor" % what)
        return t.data_ptr()
    gs = _Gaussians()
    gs.n, gs.sh_degree = int(scene.mean.shape[0]), int(scene.sh_degree)
    gs.mean, gs.scale, gs.quat = host(scene.mean, "mean"), host(scene.scale, "scale"), host(scene.quat, "quat")
    gs.opacity, gs.sh = host(scene.opacity, "opacity"), host(scene.sh, "sh")
    c, cs = cfg.c(), camera_struct(cam)
    counts = (C.c_uint32 * COUNTS_WORDS)()
    st = lib().gart_view_host(C.byref(c), C.byref(gs), C.byref(cs), host(dL_dcolor, "dL_dcolor"), host(color_out, "color_out"),
                              host(grad_out, "grad_out"), int(cap_pairs), int(cap_hits), counts,
                              _dev(arena, torch.uint8, "arena"), arena.numel(), _stream_ptr(stream))
    out = [int(v) for v in counts]
    if st != GART_OK:
        err = GartError(st, "gart_view_host")
        err.counts = out
        raise err
    return out


# ----------------------------------------------------------------------------------------- buffer plumbing
class ViewBuffers:
    """Device buffers of one view, allocated once for given capacities and reused across views."""

    def __init__(self, n, sh_degree, cam, cfg: Config, cap_pairs, cap_hits, device="cuda"):
        ts = cfg.tile_size
        self.n, self.cap_pairs, self.cap_hits = int(n), int(cap_pairs), int(cap_hits)
        H, W = int(cam.height), int(cam.width)
        T = tiles(cam, ts)
        mw = ts * ts // 32
        i32, f32, u8 = torch.int32, torch.float32, torch.uint8
        e = lambda shape, dt: torch.empty(shape, dtype=dt, device=device)
        n1, cp, ch = max(self.n, 1), max(self.cap_pairs, 1), max(self.cap_hits, 1)
        self.rect, self.cls, self.pre = e((n1, 4), i32), e((n1,), u8), e((n1, gart_pre_words(sh_degree)), f32)
        self.slot_of_gid, self.gid_of_slot = e((n1,), i32), e((n1,), i32)
        self.counts = torch.zeros(COUNTS_WORDS, dtype=i32, device=device)
        self.tile_off, self.pair_gid = e((T + 1,), i32), e((cp,), i32)
        self._geom = (n1, W, H, ts, self.cap_pairs)
        self.view = e((gart_view_bytes(*self._geom),), u8)
        self.color, self.t_final, self.hit_count = e((H, W, 3), f32), e((H, W), f32), e((H, W), i32)
        self.lt = e((ch, 4), f32)
        self.ray_off, self.ray_gid, self.ray_slot = e((H * W + 1,), i32), e((ch,), i32), e((ch,), i32)
        self.grad = e((n1, GRAD_WORDS), f32)
        self.workspace = e((gart_workspace_bytes(n1, W, H, ts, cap_pairs, cap_hits),), u8)

    def view_array(self, name):
        """One named private array of the view block as an int32 tensor (a view into the block; tests and diagnostics)."""
        off, nb = gart_view_array(*self._geom, name)
        return self.view[off:off + nb].view(torch.int32)

    def bytes(self):
        return sum(t.numel() * t.element_size() for t in vars(self).values() if isinstance(t, torch.Tensor))


def run_bounds_tile_map(cfg, g, cam, buf: ViewBuffers, stream=None):
    gart_bounds(cfg, g, cam, buf.rect, buf.cls, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.counts, buf.workspace, stream)
    gart_tile_map(cfg, buf.rect, g.n, cam, buf.tile_off, buf.pair_gid, buf.cap_pairs, buf.counts, buf.workspace, stream)


def run_forward(cfg, g, cam, buf: ViewBuffers, stream=None, ray_lists=True):
    """ray_lists=False skips the per-ray ordered hit lists (needed only by the atomic baseline and by parity checks)."""
    gart_forward(cfg, g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.pair_gid, buf.cap_pairs, buf.color,
                 buf.t_final, buf.hit_count, buf.lt, buf.cap_hits, buf.ray_off, buf.ray_gid if ray_lists else None,
                 buf.ray_slot if ray_lists else None, buf.view, buf.counts, buf.workspace, stream)


def run_backward(cfg, g, cam, buf: ViewBuffers, dL_dcolor, grad=None, stream=None):
    gart_backward(cfg, g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view, buf.cap_pairs, buf.lt, dL_dcolor,
                  buf.grad if grad is None else grad, buf.counts, buf.workspace, stream)


def run_backward_tile(cfg, g, cam, buf: ViewBuffers, dL_dcolor, grad=None, stream=None):
    """cfg.lt_layout must be LT_TILE_MAJOR and the forward must have run with the same cfg."""
    gart_backward_tile(cfg, g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view, buf.cap_pairs, buf.lt,
                       dL_dcolor, buf.grad if grad is None else grad, buf.counts, buf.workspace, stream)


def run_backward_warp(cfg, g, cam, buf: ViewBuffers, dL_dcolor, grad=None, stream=None):
    gart_backward_warp(cfg, g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view, buf.cap_pairs, buf.lt,
                       dL_dcolor, buf.grad if grad is None else grad, buf.counts, buf.workspace, stream)


def run_backward_atomic(cfg, g, cam, buf: ViewBuffers, dL_dcolor, grad, stream=None):
    gart_backward_atomic(cfg, g, cam, buf.pre, buf.slot_of_gid, buf.ray_off, buf.ray_gid, buf.ray_slot, buf.lt, dL_dcolor,
                         grad, buf.counts, stream)


def run_backward_hybrid(cfg, g, cam, buf: ViewBuffers, dL_dcolor, grad=None, stream=None):
    """cfg.lt_format must be 1, cfg.lt_layout LT_TILE_MAJOR, and the forward must have run with the same cfg and the ray lists."""
    gart_backward_hybrid(cfg, g, cam, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.tile_off, buf.view, buf.cap_pairs, buf.lt,
                         buf.ray_off, buf.ray_gid, dL_dcolor, buf.grad if grad is None else grad, buf.counts, buf.workspace, stream)


def size_view(cfg, g, cam, slack=1.0, device="cuda"):
    """Run bounds + tile map with a probing allocation and return (cap_pairs, cap_hits): the exact pair
    count and a capacity that always holds the intermediate buffer (sum of rectangle areas plus the
    worst-case padding of its interleaved layout), each times `slack`.  Two host round trips; meant for
    set-up, not for the steady state."""
    probe = ViewBuffers(g.n, g.sh_degree, cam, cfg, 0, 0, device)
    run_bounds_tile_map(cfg, g, cam, probe)
    cnt = gart_read_counts(probe.counts)
    P = cnt[CNT_PAIRS]
    S = cnt[CNT_SLOTS_LO] | (cnt[CNT_SLOTS_HI] << 32)
    # padding of the interleaved layouts: a tile pads by less than 32 x its largest hit count (tile_size^2 at most), a
    # super-tile of the primitive-major layout by less than 32 x 1024 (the exact need is the LT_SLOTS count after the forward)
    ns = -(-int(cam.width) // 16) * -(-int(cam.height) // 16)
    pad = max(32 * cfg.tile_size ** 2 * min(tiles(cam, cfg.tile_size), P), 32 * 1024 * min(ns, P))
    return int(P * slack) + 1, int(S * slack) + pad + 1
