"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

import paper_2608_17298_b200.gart as G

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "gart.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gart_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    from paper_2608_17298_b200 import build
    build.build()
    L = G.lib()
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(G.EXPORTS)


def test_host_only_queries():
    assert G.gart_mask_words(8) == 2 and G.gart_mask_words(16) == 8
    assert [G.gart_pre_words(d) for d in range(4)] == [32, 32, 32, 32]   # evaluation record 20 + quaternion, scale, opacity 8 + rectangle 4
    # accumulation records: 60 words per Gaussian in two arrays, each rounded up to 256 bytes
    assert G.gart_backward_workspace_bytes(1000) == 64_000 + 176_128 and G.gart_bounds_workspace_bytes(1000) > 80_000
    assert G.lib().gart_status_string(0) == b"ok" and G.lib().gart_status_string(2) == b"workspace too small"
    a = G.gart_tile_map_workspace_bytes(1000, 640, 480, 8, 10_000)
    b = G.gart_tile_map_workspace_bytes(1000, 640, 480, 8, 20_000)
    assert 0 < a < b and a % 256 == 0
    f1 = G.gart_forward_workspace_bytes(640, 480, 8, 10_000, 100_000)
    f2 = G.gart_forward_workspace_bytes(640, 480, 8, 10_000, 200_000)
    assert abs((f2 - f1) - 100_000 * 40) <= 4 * 256    # 40 bytes of scratch per hit of capacity (+- alignment)
    assert G.gart_view_host_arena_bytes(1000, 3, 640, 480, 8, 10_000, 100_000) > f1
    # one query for the whole view: the largest of the four
    assert G.gart_workspace_bytes(1000, 640, 480, 8, 10_000, 100_000) == max(
        f1, a, G.gart_bounds_workspace_bytes(1000), G.gart_backward_hybrid_workspace_bytes(1000, 3))
    assert G.gart_backward_hybrid_workspace_bytes(1000, 3) == G.gart_backward_workspace_bytes(1000) + 1000 * 48 * 4
    assert G.gart_backward_hybrid_workspace_bytes(1000, 0) == G.gart_backward_workspace_bytes(1000) + 16128   # 1000 rows of 4 words, to 256 bytes
    # the view block: grows with the pair capacity; its named arrays lie inside it, 256-byte aligned, in order
    v1, v2 = G.gart_view_bytes(1000, 640, 480, 8, 10_000), G.gart_view_bytes(1000, 640, 480, 8, 20_000)
    assert 0 < v1 < v2 and v1 % 256 == 0 and G.gart_view_bytes(1000, 640, 480, 12, 10_000) == 0
    last = -1
    for name in G.VIEW_ARRAYS:
        off, nb = G.gart_view_array(1000, 640, 480, 8, 10_000, name)
        assert off % 256 == 0 and nb > 0 and off + nb <= v1
        if name not in ("item_desc",):
            assert off > last or last < 0
        last = max(last, off)
    assert G.gart_view_array(1000, 640, 480, 8, 10_000, "pair_mask") == (0, 10_000 * 8)
    assert G.gart_view_host_arena_bytes(1000, 5, 640, 480, 8, 10_000, 100_000) == 0
