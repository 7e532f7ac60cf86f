"""gart_tile_map_static: the tile map whose scratch is a fixed array inside the library.

It serves callers that cannot allocate device memory when they call (a host that gave its whole
device budget to its own arena, a plug-in under a quota, a loop that must not touch the allocator).
The test calls it through the C ABI twice in a row -- the second call finds the first call's
leftovers in the shared array -- and requires exactly the outputs of gart_tile_map, which are
integers: tile offsets, pair lists and the counts block must be identical; the same outputs are
compared with the oracle's tile map, and the device's free memory must be the same before and
after the second call (nothing was allocated).  It also checks that a problem too large for the
fixed array is refused with a clear status.
"""
import numpy as np
import pytest
import torch

import gart_scenes as gs
import paper_2608_17298_b200.gart as G
from oracle import gart_oracle as orc

pytestmark = pytest.mark.gpu


def _tile_maps(scene, cam, cfg):
    g = G.Gaussians.from_numpy(scene)
    P, _ = G.size_view(cfg, g, cam)
    buf = G.ViewBuffers(g.n, g.sh_degree, cam, cfg, P, 1)
    # reference: the existing entry point with a caller workspace
    G.run_bounds_tile_map(cfg, g, cam, buf)
    torch.cuda.synchronize()
    ref = (buf.tile_off.cpu().numpy().copy(), buf.pair_gid.cpu().numpy()[:P - 1].copy(), G.gart_read_counts(buf.counts))
    # the entry point under test: same rectangles, outputs into fresh arrays, no workspace argument
    tile_off = torch.full_like(buf.tile_off, -1)
    pair_gid = torch.full_like(buf.pair_gid, -1)
    G.gart_bounds(cfg, g, cam, buf.rect, buf.cls, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.counts, buf.workspace)
    G.gart_tile_map_static(cfg, buf.rect, g.n, cam, tile_off, pair_gid, P, buf.counts)
    torch.cuda.synchronize()
    got = (tile_off.cpu().numpy(), pair_gid.cpu().numpy()[:P - 1], G.gart_read_counts(buf.counts))
    # once more into the same arrays: the address of the fixed array is known by now, so the call must not touch the allocator
    free0 = torch.cuda.mem_get_info()[0]
    G.gart_tile_map_static(cfg, buf.rect, g.n, cam, tile_off, pair_gid, P, buf.counts)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert np.array_equal(tile_off.cpu().numpy(), got[0]) and np.array_equal(pair_gid.cpu().numpy()[:P - 1], got[1])
    # and the oracle's tile map of the oracle's own rectangles (identical unless a rectangle edge lies within 1e-9 of a pixel centre)
    osc = orc.OracleScene.from_scene(scene)
    rect, cls, margin = orc.bounds(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32)
    if (margin > 1e-9).all():
        o_off, o_gid, _ = orc.tile_map(rect, cam.width, cam.height, cfg.tile_size)
        assert np.array_equal(got[0].astype(np.int64), np.asarray(o_off, dtype=np.int64))
        assert np.array_equal(got[1].astype(np.int64), np.asarray(o_gid, dtype=np.int64)[:P - 1])
    return ref, got


def test_static_scratch_tile_map_matches_twice_in_a_row():
    cases = [(gs.config_cluster(n=20_000, width=320, height=240), 8), (gs.config_tiny(n=300, sh_degree=1, seed=4), 16)]
    for (scene, cams), ts in cases:                     # second call: different sizes, stale scratch from the first
        ref, got = _tile_maps(scene, cams[0], G.Config(tile_size=ts))
        assert ref[2][G.CNT_PAIRS] > 100 and ref[2][G.CNT_ERROR] == 0
        assert np.array_equal(ref[0], got[0])
        assert np.array_equal(ref[1], got[1])
        assert ref[2] == got[2]


def test_static_scratch_refuses_oversized_problems():
    scene, cams = gs.config_tiny(n=64)
    cam, cfg = cams[0], G.Config()
    g = G.Gaussians.from_numpy(scene)
    buf = G.ViewBuffers(g.n, g.sh_degree, cam, cfg, 16, 1)
    G.gart_bounds(cfg, g, cam, buf.rect, buf.cls, buf.pre, buf.slot_of_gid, buf.gid_of_slot, buf.counts, buf.workspace)
    assert G.gart_tile_map_workspace_bytes(g.n, cam.width, cam.height, 8, 4_000_000) > G.TILE_MAP_STATIC_BYTES
    with pytest.raises(G.GartError) as e:
        G.gart_tile_map_static(cfg, buf.rect, g.n, cam, buf.tile_off, buf.pair_gid, 4_000_000, buf.counts)
    assert e.value.status == 2        # GART_ERR_WORKSPACE_TOO_SMALL, nothing was launched
    torch.cuda.synchronize()
