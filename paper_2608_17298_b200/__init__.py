"""B200-native (sm_100a) hot path of primitive-centric ray-traced Gaussian rendering.

``paper_2608_17298_b200.gart`` binds the C ABI of ``libgart.so`` (declared in ``include/gart.h``):
gart_bounds, gart_tile_map, gart_forward, gart_backward and the pixel-centric baseline
gart_backward_atomic.  Build the library with ``python -m paper_2608_17298_b200.build``.
"""
from . import gart  # noqa: F401
from .gart import (Config, Gaussians, GartError, ViewBuffers, gart_backward, gart_backward_atomic, gart_bounds,  # noqa: F401
                   gart_forward, gart_forward_workspace_bytes, gart_mask_words, gart_read_counts, gart_tile_map,
                   gart_tile_map_workspace_bytes, gart_view_host, gart_view_host_arena_bytes)
