"""Helpers of the GPU parity tests: run the CUDA path, run the oracle, compare.

Comparison protocol
-------------------
Integer artefacts (rectangles, classes, tile lists) must be identical, except for a Gaussian
whose float64 decision margin is below 1e-9 (a pixel-centre exactly on a bound).

Hit decisions and the per-ray order are taken in fp32 on the GPU and in float64 by the oracle.
A decision may differ only inside a guard band: a hit present on one side only must have
|ln(alpha / alpha_min)| < BAND_HIT in float64, and the GPU's order of two consecutive hits
may differ from the (t*, id) order only if their float64 t* agree within BAND_ORDER (relative).
Such cases are counted and reported; the oracle then composites and differentiates the GPU's
own hit lists ("replay"), so that colour and gradient tolerances apply to every ray.
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2608_17298_b200.gart as G
from oracle import gart_oracle as orc

BAND_HIT = 2e-4
BAND_ORDER = 2e-5


def to_np(t):
    return t.detach().cpu().numpy()


def u32(a):
    return a.view(np.uint32) if a.dtype == np.int32 else a


def _view_arrays(buf, names, P, mw):
    out = {}
    for nme in names:
        a = u32(to_np(buf.view_array(nme)))
        if nme in ("pair_mask", "rank_mask", "gm_mask"):
            a = a.reshape(-1, mw)[:P]
        elif nme == "item_desc":
            a = a.reshape(-1, 4)
        elif nme in ("pair_order", "rank_sid", "rank_gstart", "pair_gpos", "gm_ltb"):
            a = a[:P]
        out[nme] = a.copy()
    return out


GUARD_BYTES = 1024
GUARDED = ("rect", "cls", "pre", "slot_of_gid", "gid_of_slot", "tile_off", "pair_gid", "view", "color", "t_final", "hit_count", "lt",
           "ray_off", "ray_gid", "ray_slot", "grad", "workspace")


def guard_buffers(buf):
    """Re-seat every device buffer of the view between two guard zones of GUARD_BYTES filled with a pattern (the buffer
    keeps its size, type and 256-byte alignment).  Returns the backing tensors for check_guards."""
    backing = {}
    for nme in GUARDED:
        t = getattr(buf, nme)
        nb = t.numel() * t.element_size()
        flat = torch.full((nb + 2 * GUARD_BYTES,), 0xA5, dtype=torch.uint8, device=t.device)
        setattr(buf, nme, flat[GUARD_BYTES:GUARD_BYTES + nb].view(t.dtype).view(t.shape))
        backing[nme] = (flat, nb)
    return backing


def check_guards(backing):
    """No kernel wrote in front of or behind any buffer."""
    for nme, (flat, nb) in backing.items():
        assert bool((flat[:GUARD_BYTES] == 0xA5).all()) and bool((flat[GUARD_BYTES + nb:] == 0xA5).all()), ("guard zone of %s overwritten" % nme)


def run_gpu(scene, cam, cfg: G.Config, dL_dC, cap_pairs=None, cap_hits=None, atomic=True, guard=False):
    """Full device path for one view; returns numpy copies of every output.  The view runs in the primitive-major LT
    layout (gart_backward); with atomic=True the other backward variants follow: the pixel-centric baseline on the
    same buffers, then the forward again in the tile-major layout for the block-per-tile pass, the warp-per-pair pass
    and the hybrid pass, and the forward with 8-byte entries for gart_backward on them."""
    import dataclasses
    cfg = dataclasses.replace(cfg, lt_layout=G.LT_PRIMITIVE_MAJOR)
    g = G.Gaussians.from_numpy(scene)
    if cap_pairs is None or cap_hits is None:
        P, S = G.size_view(cfg, g, cam, slack=1.0)
        cap_pairs = P if cap_pairs is None else cap_pairs
        cap_hits = S if cap_hits is None else cap_hits
    buf = G.ViewBuffers(g.n, g.sh_degree, cam, cfg, cap_pairs, cap_hits)
    backing = guard_buffers(buf) if guard else None
    buf.grad.fill_(float("nan"))          # every record must be written by the backward pass
    dl = torch.from_numpy(np.ascontiguousarray(dL_dC, dtype=np.float32)).cuda()
    G.run_bounds_tile_map(cfg, g, cam, buf)
    G.run_forward(cfg, g, cam, buf)
    G.run_backward(cfg, g, cam, buf, dl)
    counts = G.gart_read_counts(buf.counts)
    out = {"counts": counts, "buf": buf, "g": g, "dl": dl}
    P, H = counts[G.CNT_PAIRS], counts[G.CNT_HITS]
    mw = cfg.tile_size ** 2 // 32
    out["rect"], out["cls"] = to_np(buf.rect)[:g.n], to_np(buf.cls)[:g.n]
    out["tile_off"] = u32(to_np(buf.tile_off))
    if counts[G.CNT_ERROR]:
        if guard:
            check_guards(backing)
        return out
    out["pair_gid"] = u32(to_np(buf.pair_gid))[:P]
    out["slot_of_gid"], out["gid_of_slot"] = u32(to_np(buf.slot_of_gid))[:g.n], u32(to_np(buf.gid_of_slot))[:g.n]
    out.update(_view_arrays(buf, ["pair_mask", "pair_order", "rank_sid", "rank_mask", "pair_gpos", "gpair_off", "gm_mask", "gm_ltb",
                                  "item_desc", "item_gstart", "st_off", "st_lt_base", "info"], P, mw))
    out["color"], out["t_final"] = to_np(buf.color), to_np(buf.t_final)
    out["hit_count"] = u32(to_np(buf.hit_count))
    out["ray_off"] = u32(to_np(buf.ray_off))
    out["ray_gid"] = u32(to_np(buf.ray_gid))[:H]
    out["ray_slot"] = u32(to_np(buf.ray_slot))[:H]
    out["lt"] = to_np(buf.lt)[:counts[G.CNT_LT_SLOTS]]
    out["grad"] = to_np(buf.grad)[:g.n].copy()
    if atomic:
        ga = torch.full_like(buf.grad, float("nan"))
        G.run_backward_atomic(cfg, g, cam, buf, dl, ga)
        torch.cuda.synchronize()
        out["grad_atomic"] = to_np(ga)[:g.n]
        gv = torch.full_like(buf.grad, float("nan"))
        G.run_backward_atomic(dataclasses.replace(cfg, atomic_mode=1), g, cam, buf, dl, gv)     # the same sums as vector reductions
        torch.cuda.synchronize()
        out["grad_atomic_vec"] = to_np(gv)[:g.n]
        # ---- tile-major layout: block-per-tile pass and warp-per-pair pass (same buffers, the forward again)
        cfg_t = dataclasses.replace(cfg, lt_layout=G.LT_TILE_MAJOR)
        G.run_forward(cfg_t, g, cam, buf)
        for key, fn in (("grad_tile", G.run_backward_tile), ("grad_warp", G.run_backward_warp)):
            gt = torch.full_like(buf.grad, float("nan"))
            fn(cfg_t, g, cam, buf, dl, gt)
            torch.cuda.synchronize()
            out[key] = to_np(gt)[:g.n]
        ct = G.gart_read_counts(buf.counts)
        assert ct[G.CNT_ERROR] == 0 and ct[G.CNT_HITS] == H
        tile = _view_arrays(buf, ["pair_mask", "pair_order", "rank_sid", "rank_mask", "rank_gstart", "tile_lt_base"], P, mw)
        tile["ray_slot"] = u32(to_np(buf.ray_slot))[:H].copy()
        tile["lt"] = to_np(buf.lt)[:ct[G.CNT_LT_SLOTS]].copy()
        tile["lt_slots"] = ct[G.CNT_LT_SLOTS]
        out["tile"] = tile
        # the other outputs of the forward do not depend on the LT layout
        assert np.array_equal(to_np(buf.color), out["color"]) and np.array_equal(u32(to_np(buf.ray_gid))[:H], out["ray_gid"])
        assert np.array_equal(tile["pair_mask"], out["pair_mask"])
        if cfg.max_hits == 0 and cfg.t_min == 0 and cfg.alpha_max >= 1 and cfg.kernel_degree == 2:   # (the hybrid backward re-derives every alpha in its pixel pass: no cap, early end or clamp, Gaussian response)
            # hybrid backward: the forward again with 4-byte LT entries
            cfg_h = dataclasses.replace(cfg_t, lt_format=1)
            G.run_forward(cfg_h, g, cam, buf)
            gh = torch.full_like(buf.grad, float("nan"))
            G.run_backward_hybrid(cfg_h, g, cam, buf, dl, gh)
            torch.cuda.synchronize()
            assert G.gart_read_counts(buf.counts)[G.CNT_ERROR] == 0
            out["grad_hybrid"] = to_np(gh)[:g.n]
            assert np.array_equal(to_np(buf.color), out["color"]) and np.array_equal(u32(to_np(buf.ray_gid))[:H], out["ray_gid"])
        # 8-byte LT entries (four halves per hit): the block-per-tile pass on them (tile-major layout)
        cfg_8t = dataclasses.replace(cfg_t, lt_format=2)
        G.run_forward(cfg_8t, g, cam, buf)
        g8 = torch.full_like(buf.grad, float("nan"))
        G.run_backward_tile(cfg_8t, g, cam, buf, dl, g8)
        torch.cuda.synchronize()
        assert G.gart_read_counts(buf.counts)[G.CNT_ERROR] == 0
        out["grad_lt16"] = to_np(g8)[:g.n]
        out["lt16"] = to_np(buf.lt).reshape(-1).view(np.uint16)[:4 * tile["lt_slots"]].reshape(-1, 4).copy()
        assert np.array_equal(to_np(buf.color), out["color"]) and np.array_equal(u32(to_np(buf.ray_slot))[:H], tile["ray_slot"])
    if guard:
        torch.cuda.synchronize()
        check_guards(backing)
    return out


def check_maps(scene, cam, cfg: G.Config, gpu):
    """Rectangles, classes and tile lists against the oracle (bit-exact outside the 1e-9 margin)."""
    osc = orc.OracleScene.from_scene(scene)
    rect, cls, margin = orc.bounds(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32, kernel_degree=cfg.kernel_degree)
    safe = margin > 1e-9
    assert safe.mean() > 0.999
    assert np.array_equal(gpu["cls"][safe], cls[safe])
    assert np.array_equal(gpu["rect"][safe], rect[safe])
    same = np.array_equal(gpu["rect"], rect)
    # tile lists follow from the rectangles: check them against the oracle on the GPU's rectangles
    # (identical to the oracle's own unless a sub-1e-9 margin flipped an edge)
    tile_off, pair_gid, slots = orc.tile_map(gpu["rect"], cam.width, cam.height, cfg.tile_size)
    assert np.array_equal(gpu["tile_off"], tile_off)
    assert np.array_equal(gpu["pair_gid"], pair_gid)
    c = gpu["counts"]
    assert c[G.CNT_PAIRS] == len(pair_gid)
    assert (c[G.CNT_SLOTS_LO] | (c[G.CNT_SLOTS_HI] << 32)) == slots
    assert c[G.CNT_VISIBLE] == int((gpu["rect"][:, 2] >= gpu["rect"][:, 0]).sum())
    return {"rect_identical": bool(same), "n_unsafe": int((~safe).sum()), "osc": osc}


SUP = 16   # super-tile edge of the primitive-major order, pixels


def _sample_hits(cam, gpu, max_rays, seed):
    """(rays, index into the per-ray lists) of every hit, or of the hits of a random subset of rays on large views."""
    H = gpu["counts"][G.CNT_HITS]
    ray_off, hit_count = gpu["ray_off"].astype(np.int64), gpu["hit_count"].reshape(-1).astype(np.int64)
    n_rays = hit_count.size
    if H > 5_000_000:
        rsel = np.sort(np.random.default_rng(seed).choice(n_rays, size=max_rays, replace=False))
    else:
        rsel = np.arange(n_rays)
    cnt = hit_count[rsel]
    idx = np.repeat(ray_off[rsel], cnt) + (np.arange(cnt.sum()) - np.repeat(np.cumsum(cnt) - cnt, cnt))
    return np.repeat(rsel, cnt), idx


def _locate_pairs(cam, cfg, gpu, rays, gids):
    """Pair index (in the tile-major pair list) of every (ray, Gaussian) hit, and the hit's index among the set bits of the
    pair's mask (pixel order)."""
    ts = cfg.tile_size
    tiles_x = -(-cam.width // ts)
    tile_off = gpu["tile_off"].astype(np.int64)
    n_tile = np.diff(tile_off)
    tile_of_pair = np.repeat(np.arange(n_tile.size), n_tile)
    tile = (rays // cam.width) // ts * tiles_x + (rays % cam.width) // ts
    pair_gid = gpu["pair_gid"].astype(np.int64)
    P = pair_gid.size
    mul = int(pair_gid.max()) + 1 if P else 1
    key = tile_of_pair * mul + pair_gid                      # ascending: ids ascend inside a tile
    want = tile * mul + gids
    pair = np.searchsorted(key, want)
    assert np.array_equal(key[pair], want)
    px = (rays % cam.width) % ts + ((rays // cam.width) % ts) * ts
    words = gpu["pair_mask"][pair]                                  # [h, MW]
    w_idx, b_idx = px // 32, px % 32
    word = words[np.arange(pair.size), w_idx].astype(np.uint64)
    assert np.all((word >> b_idx.astype(np.uint64)) & np.uint64(1))   # the hit pixel is set in the pair's mask
    below = np.bitwise_count(word & ((np.uint64(1) << b_idx.astype(np.uint64)) - np.uint64(1))).astype(np.int64)
    for q in range(words.shape[1]):
        below += np.where(q < w_idx, np.bitwise_count(words[:, q]).astype(np.int64), 0)
    return pair, below, tile


def all_distinct_below(a, bound):
    """True if the non-negative integers of `a` are pairwise distinct and all below `bound` (a flag per value: linear time)."""
    a = np.asarray(a).astype(np.int64, copy=False)
    if a.size == 0:
        return True
    if int(a.max()) >= bound or int(a.min()) < 0:
        return False
    seen = np.zeros(int(bound), dtype=bool)
    seen[a] = True
    return int(np.count_nonzero(seen)) == a.size


def check_structure(cam, cfg: G.Config, gpu, max_rays=20000, seed=0):
    """Properties that hold at any size, checked on the whole view without the oracle (the per-hit part on a random
    subset of rays when the view has more than a few million hits): ray offsets, hit masks, slot numbering, and the
    primitive-major work lists and LT layout re-derived in numpy from rectangles and masks."""
    H = gpu["counts"][G.CNT_HITS]
    L = gpu["counts"][G.CNT_LT_SLOTS]
    ts = cfg.tile_size
    ray_off, hit_count = gpu["ray_off"].astype(np.int64), gpu["hit_count"].reshape(-1).astype(np.int64)
    assert ray_off[0] == 0 and ray_off[-1] == H and np.array_equal(np.diff(ray_off), hit_count)
    assert gpu["counts"][G.CNT_MAX_RAY_HITS] == (hit_count.max() if hit_count.size else 0)
    pc = np.bitwise_count(gpu["pair_mask"]).sum(axis=1).astype(np.int64)
    assert pc.sum() == H and L >= H
    # every hit owns exactly one slot
    slots_all = gpu["ray_slot"]
    assert slots_all.size == H and all_distinct_below(slots_all, L)
    P = pc.size
    # ---- slots: visible Gaussians in the order of the super-tile of their rectangle's corner, ids ascending inside one
    rect_ = gpu["rect"].astype(np.int64)
    vis = rect_[:, 2] >= rect_[:, 0]
    V = int(vis.sum())
    sup_x = -(-cam.width // SUP)
    key_ = (rect_[:, 1] // SUP) * sup_x + rect_[:, 0] // SUP
    want_order = np.nonzero(vis)[0][np.argsort(key_[vis], kind="stable")]
    assert np.array_equal(gpu["gid_of_slot"][:V], want_order.astype(np.uint32)) and np.all(gpu["gid_of_slot"][V:] == 0xffffffff)
    inv = np.full(rect_.shape[0], 0xffffffff, np.uint32)
    inv[want_order] = np.arange(V, dtype=np.uint32)
    assert np.array_equal(gpu["slot_of_gid"], inv)
    # ---- primitive-major pair positions: a slot's tiles row by row
    r = rect_[want_order]                                          # rectangles in slot order
    tx0, ty0, tx1, ty1 = r[:, 0] // ts, r[:, 1] // ts, r[:, 2] // ts, r[:, 3] // ts
    ntx, nty = tx1 - tx0 + 1, ty1 - ty0 + 1
    gpo = np.concatenate([[0], np.cumsum(ntx * nty)])
    assert gpo[-1] == P and np.array_equal(gpu["gpair_off"][:V + 1].astype(np.int64), gpo)
    tiles_x = -(-cam.width // ts)
    tile_off = gpu["tile_off"].astype(np.int64)
    tile_of_pair = np.repeat(np.arange(tile_off.size - 1), np.diff(tile_off))
    sl = gpu["slot_of_gid"][gpu["pair_gid"]].astype(np.int64)
    ptx, pty = tile_of_pair % tiles_x, tile_of_pair // tiles_x
    gpos = gpo[sl] + (pty - ty0[sl]) * ntx[sl] + (ptx - tx0[sl])
    assert np.array_equal(gpu["pair_gpos"].astype(np.int64), gpos) and all_distinct_below(gpos, P)
    assert np.array_equal(gpu["gm_mask"][gpos], gpu["pair_mask"])
    pc_g = np.empty(P, np.int64)
    pc_g[gpos] = pc                                                # hits per pair, by primitive-major position
    # ---- work items: a Gaussian spanning at most two super-tiles per axis is one item owned by the super-tile of its
    # corner, any other is cut into one item per super-tile it touches; emission order = slot order, pieces row by row
    sx0, sy0, sx1, sy1 = r[:, 0] // SUP, r[:, 1] // SUP, r[:, 2] // SUP, r[:, 3] // SUP
    whole = ((sx1 - sx0) <= 1) & ((sy1 - sy0) <= 1)
    nsx = np.where(whole, 1, sx1 - sx0 + 1)
    n_it = np.where(whole, 1, (sx1 - sx0 + 1) * (sy1 - sy0 + 1))
    I = int(n_it.sum())
    assert gpu["info"][0] == I
    it_slot = np.repeat(np.arange(V), n_it)
    local = np.arange(I) - np.repeat(np.cumsum(n_it) - n_it, n_it)
    it_sx, it_sy = sx0[it_slot] + local % nsx[it_slot], sy0[it_slot] + local // nsx[it_slot]
    it_whole = whole[it_slot]
    tps = SUP // ts                                                # tiles per super-tile edge
    fx = np.where(it_whole, tx0[it_slot], np.maximum(tx0[it_slot], it_sx * tps))
    lx = np.where(it_whole, tx1[it_slot], np.minimum(tx1[it_slot], it_sx * tps + tps - 1))
    fy = np.where(it_whole, ty0[it_slot], np.maximum(ty0[it_slot], it_sy * tps))
    ly = np.where(it_whole, ty1[it_slot], np.minimum(ty1[it_slot], it_sy * tps + tps - 1))
    it_ntx, it_nty = lx - fx + 1, ly - fy + 1
    gpos0 = gpo[it_slot] + (fy - ty0[it_slot]) * ntx[it_slot] + (fx - tx0[it_slot])
    # hits per item and, per pair of an item, the hits of the item's earlier pairs
    npair = it_ntx * it_nty
    pi = np.repeat(np.arange(I), npair)
    kk = np.arange(npair.sum()) - np.repeat(np.cumsum(npair) - npair, npair)
    pg = gpos0[pi] + (kk // it_ntx[pi]) * ntx[it_slot][pi] + kk % it_ntx[pi]      # primitive-major position of the item's k-th pair
    assert pg.size == P and all_distinct_below(pg, P)               # the items partition the pairs
    it_cnt = np.bincount(pi, weights=pc_g[pg], minlength=I).astype(np.int64)
    csum = np.cumsum(pc_g[pg]) - pc_g[pg]
    before = csum - np.repeat((np.cumsum(it_cnt) - it_cnt), npair)
    S_own = it_sy * sup_x + it_sx
    NS = sup_x * -(-cam.height // SUP)
    order = np.lexsort((np.arange(I), -it_cnt, S_own))              # by super-tile, then descending hits, stable
    st_off = np.concatenate([[0], np.cumsum(np.bincount(S_own, minlength=NS))])
    assert np.array_equal(gpu["st_off"].astype(np.int64), st_off)
    desc = gpu["item_desc"][:I].astype(np.int64)
    assert np.array_equal(desc[:, 0], it_slot[order]) and np.array_equal(desc[:, 1], gpos0[order])
    dims = ntx[it_slot] | (it_ntx << 16) | (it_nty << 20) | ((fx - it_sx * tps) << 24) | ((fy - it_sy * tps) << 28)
    assert np.array_equal(desc[:, 2], dims[order])
    assert np.array_equal(desc[:, 3], (it_cnt | (it_whole.astype(np.int64) << 16))[order])
    # groups of 32 ranks inside a super-tile occupy 32 x (largest count, rounded up to even) entries
    So, co = S_own[order], it_cnt[order]
    rank = np.arange(I) - st_off[So]
    first = rank % 32 == 0
    gsize = 32 * (co[first] + (co[first] & 1))
    gS = So[first]
    gstart = np.cumsum(gsize) - gsize                               # super-tiles are laid out one after the other
    assert np.array_equal(gpu["item_gstart"][:I].astype(np.int64), np.repeat(gstart, np.diff(np.r_[np.nonzero(first)[0], I])))
    st_len = np.bincount(gS, weights=gsize, minlength=NS).astype(np.int64)
    assert np.array_equal(gpu["st_lt_base"].astype(np.int64), np.concatenate([[0], np.cumsum(st_len)])) and st_len.sum() == L
    # LT entry of an item's e-th hit (e counts through the item's pairs in turn): entries go two by two, the two of a
    # lane share a 32-byte sector, the 32 lanes' sectors of the same pair of entries are consecutive
    def slot_of(gs, lane, e):
        return gs + (e >> 1) * 64 + 2 * lane + (e & 1)
    pos_of_item = np.empty(I, np.int64)
    pos_of_item[order] = np.arange(I)
    g_of_item = gpu["item_gstart"][:I].astype(np.int64)[pos_of_item]
    lane_of_item = rank[pos_of_item] % 32
    ltb = np.empty(P, np.int64)
    ltb[pg] = slot_of(g_of_item[pi], lane_of_item[pi], before)
    assert np.array_equal(gpu["gm_ltb"].astype(np.int64), ltb)
    item_of_gpos = np.empty(P, np.int64)
    item_of_gpos[pg] = pi
    before_g = np.empty(P, np.int64)
    before_g[pg] = before
    # ---- per hit: on all rays, or on a random subset of them
    rays, idx = _sample_hits(cam, gpu, max_rays, seed)
    slots = gpu["ray_slot"][idx].astype(np.int64)
    gids = gpu["ray_gid"][idx].astype(np.int64)
    pair, below, _ = _locate_pairs(cam, cfg, gpu, rays, gids)
    it = item_of_gpos[gpos[pair]]                                   # the e-th hit of a pair: its e-th set mask bit in pixel order
    assert np.array_equal(slots, slot_of(g_of_item[it], lane_of_item[it], before_g[gpos[pair]] + below))
    # LT: word 3 is the blending weight T alpha in (0, 1) with the three clamp flags in its low mantissa
    # bits; the vector part is finite.  (The values themselves are checked against the oracle's entries.)
    used = gpu["lt"][slots]
    bits = np.ascontiguousarray(used).view(np.uint32)
    wgt = (bits[:, 3] & np.uint32(0xFFFFFFF0)).view(np.float32)
    assert np.all(np.isfinite(used)) and np.all(wgt >= 0) and np.all(wgt < 1.0)
    # ... and the entry names its pixel inside the 32 x 32 window of the item's owner: ten bits spread over the low
    # mantissa bits of the four words
    pix = (bits[:, 0] & 7) | ((bits[:, 1] & 7) << 3) | ((bits[:, 2] & 7) << 6) | ((bits[:, 3] & 8) << 6)
    own = S_own[it]
    wx = rays % cam.width - (own % sup_x) * SUP
    wy = rays // cam.width - (own // sup_x) * SUP
    assert np.all((wx >= 0) & (wx < 2 * SUP) & (wy >= 0) & (wy < 2 * SUP))
    # (a hit that is not composited -- behind a cap or behind the end of its ray -- has zero words, a sign or flag bit at
    # most, and pixel index 0: it adds exactly nothing whatever pixel it names)
    dead = np.all((bits & np.uint32(0x7FFFFFF0)) == 0, axis=1)
    assert np.all((pix.astype(np.int64) == wy * 2 * SUP + wx) | (dead & (pix == 0)))
    if cfg.max_hits > 0:
        capped = idx - ray_off[rays] >= cfg.max_hits
        assert np.all(dead[capped]) and (cfg.t_min > 0 or not dead[~capped].any())
    assert np.all(np.isfinite(gpu["color"])) and np.all(np.isfinite(gpu["grad"]))
    return {"items": I, "whole_share": float(whole.mean()) if V else 1.0, "lt_padding": float(L) / max(H, 1)}


def check_structure_tile(cam, cfg: G.Config, gpu, max_rays=20000, seed=0):
    """The tile-major work lists and LT layout (the forward run with lt_layout = tile-major: gpu["tile"])."""
    t = gpu["tile"]
    H, L = gpu["counts"][G.CNT_HITS], t["lt_slots"]
    pc = np.bitwise_count(t["pair_mask"]).sum(axis=1).astype(np.int64)
    slots_all = t["ray_slot"]
    assert slots_all.size == H and all_distinct_below(slots_all, L) and L >= H
    tile_off, base = gpu["tile_off"].astype(np.int64), t["tile_lt_base"].astype(np.int64)
    assert base[0] == 0 and base[-1] == L and np.all(np.diff(base) >= 0)
    n_tile = np.diff(tile_off)
    P = pc.size
    tile_of_pair = np.repeat(np.arange(n_tile.size), n_tile)
    # pair_order: a permutation of each tile's pairs in descending hit count, stable
    order = t["pair_order"].astype(np.int64)
    seen = np.zeros(P, bool)
    seen[order] = True
    assert seen.all()
    assert np.array_equal(tile_of_pair[order], tile_of_pair)
    rank = np.arange(P) - tile_off[tile_of_pair]                 # rank of position q within its tile
    po = pc[order]
    same_tile = tile_of_pair[1:] == tile_of_pair[:-1]
    assert np.all((po[:-1] >= po[1:]) | ~same_tile)
    assert np.all((order[:-1] < order[1:]) | (po[:-1] != po[1:]) | ~same_tile)
    # copies in rank order
    assert np.array_equal(t["rank_sid"], gpu["slot_of_gid"][gpu["pair_gid"][order]])
    assert np.array_equal(t["rank_mask"], t["pair_mask"][order])
    # rank_gstart: start of the 32-rank group; a group spans 32 x its largest (= first) count
    gs_ = t["rank_gstart"].astype(np.int64)                   # by position in rank order
    first = rank % 32 == 0
    grp_start, grp_tile, grp_size = gs_[first], tile_of_pair[first], 32 * po[first]
    assert np.array_equal(np.repeat(grp_start, np.diff(np.r_[np.nonzero(first)[0], P])), gs_)
    slot0 = np.empty(P, np.int64)
    slot0[order] = gs_ + rank % 32                               # per pair: first LT entry relative to the tile
    nxt_same = grp_tile[1:] == grp_tile[:-1]
    assert np.all((grp_start[1:] == grp_start[:-1] + grp_size[:-1]) | ~nxt_same)
    assert np.all(grp_start[np.r_[True, ~nxt_same]] == 0)
    last_of_tile = np.r_[~nxt_same, True]
    tile_len = np.zeros(n_tile.size, np.int64)
    tile_len[grp_tile[last_of_tile]] = (grp_start + grp_size)[last_of_tile]
    assert np.array_equal(tile_len, np.diff(base))
    rays, idx = _sample_hits(cam, gpu, max_rays, seed)
    slots = t["ray_slot"][idx].astype(np.int64)
    gids = gpu["ray_gid"][idx].astype(np.int64)
    pair, below, tile = _locate_pairs(cam, cfg, gpu, rays, gids)
    rel = slots - base[tile]
    assert np.all(rel >= 0) and np.all(slots < base[tile + 1])
    assert np.array_equal(rel, slot0[pair] + 32 * below)
    # the entries are the same numbers in both layouts, up to the low mantissa bits in which the primitive-major
    # entries carry their pixel index
    a = np.ascontiguousarray(t["lt"][slots]).view(np.uint32)
    b = np.ascontiguousarray(gpu["lt"][gpu["ray_slot"][idx].astype(np.int64)]).view(np.uint32)
    keep = np.array([0xFFFFFFF8, 0xFFFFFFF8, 0xFFFFFFF8, 0xFFFFFFF7], np.uint32)
    assert np.array_equal(a & keep, b & keep)


def _lists_for(ray_off, gid, rays):
    """Sub-lists of the selected rays as (ray_off_full [n_rays+1], gid) with other rays empty."""
    n_rays = ray_off.size - 1
    cnt = np.zeros(n_rays, dtype=np.int64)
    cnt[rays] = (ray_off[rays + 1] - ray_off[rays]).astype(np.int64)
    new_off = np.zeros(n_rays + 1, dtype=np.uint64)
    new_off[1:] = np.cumsum(cnt)
    idx = np.concatenate([np.arange(ray_off[r], ray_off[r + 1], dtype=np.int64) for r in rays]) if len(rays) else np.zeros(0, np.int64)
    return new_off, gid[idx].astype(np.uint32)


def check_hits_and_replay(osc, cam, cfg: G.Config, gpu, dL_dC, pixel_mask=None, mode=orc.BRUTE):
    """Compare the GPU's per-ray hit lists with the oracle's on the selected rays, under the guard
    band protocol; then replay the GPU's lists through the oracle.  Returns the replayed view's
    colour, t_final, gradient, gradient conditioning and statistics."""
    n_rays = cam.width * cam.height
    sel = np.arange(n_rays) if pixel_mask is None else np.nonzero(pixel_mask.reshape(-1))[0]
    v = orc.View(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32, bg=cfg.background, kernel_degree=cfg.kernel_degree)
    v.find_hits(mode, pixel_mask)
    o_off, o_gid, o_t, o_alpha = v.hits()
    g_off, g_gid = gpu["ray_off"].astype(np.int64), gpu["ray_gid"]
    o_off = o_off.astype(np.int64)
    stats = {"rays": int(sel.size), "oracle_hits": int(o_off[-1]), "band_hit": 0, "band_order": 0}
    g_cnt, o_cnt = g_off[sel + 1] - g_off[sel], o_off[sel + 1] - o_off[sel]
    # fast path: concatenate selected lists and compare wholesale
    g_new_off, g_sel_gid = _lists_for(gpu["ray_off"].astype(np.int64), g_gid, sel)
    identical = np.array_equal(g_cnt, o_cnt) and np.array_equal(g_sel_gid, o_gid)
    band_bound = {}      # ray -> bound on what its guard-band decisions can move its colour by (see below)
    if not identical:
        amin = cfg.alpha_min_f32
        cb = 0.5 + np.abs(osc.sh).max(axis=2).sum(axis=1)      # |colour| of a Gaussian is at most this (|Y_k| <= 1)
        for k, r in enumerate(sel):
            gl = g_gid[g_off[r]:g_off[r + 1]]
            ol = o_gid[o_off[r]:o_off[r + 1]]
            if gl.size == ol.size and np.array_equal(gl, ol):
                continue
            gs, os_ = set(gl.tolist()), set(ol.tolist())
            for gid in gs ^ os_:
                alpha, t = v.eval_pair(int(r), int(gid))
                assert abs(np.log(alpha / amin)) < BAND_HIT or (alpha >= amin and abs(t) < 1e-6), \
                    ("hit decision differs outside the guard band", int(r), int(gid), alpha, t)
                stats["band_hit"] += 1
                # a hit more or less moves the colour by T alpha (c - colour behind): at most alpha (|c| + largest colour)
                band_bound[int(r)] = band_bound.get(int(r), 0.0) + alpha * (cb[gid] + max(cb[gl].max(initial=0.0), float(np.max(np.abs(cfg.background)))))
            # order of the GPU list must be non-decreasing in float64 t* up to the band
            ts_ = np.array([v.eval_pair(int(r), int(gid))[1] for gid in gl])
            if ts_.size > 1:
                viol = ts_[:-1] > ts_[1:] * (1 + BAND_ORDER)
                assert not viol.any(), ("order differs outside the guard band", int(r))
                eq = np.abs(ts_[:-1] - ts_[1:]) <= BAND_ORDER * np.abs(ts_[1:])
                # equal within the band: either order accepted; exact ties must ascend in id
                exact = ts_[:-1] == ts_[1:]
                assert np.all(gl[:-1][exact] < gl[1:][exact])
                common = [x for x in gl.tolist() if x in os_]
                common_o = [x for x in ol.tolist() if x in gs]
                stats["band_order"] += int(common != common_o)
                if common != common_o:
                    # two hits composited the other way round move the colour by T alpha_i alpha_j (c_i - c_j)
                    pos_o = {x: i for i, x in enumerate(common_o)}
                    al = {int(x): v.eval_pair(int(r), int(x))[0] for x in common}
                    b = 0.0
                    for i in range(len(common)):
                        for j in range(i + 1, len(common)):
                            if pos_o[common[i]] > pos_o[common[j]]:
                                b += al[common[i]] * al[common[j]] * (cb[common[i]] + cb[common[j]])
                    band_bound[int(r)] = band_bound.get(int(r), 0.0) + b
    stats["identical_lists"] = bool(identical)
    stats["band_rays"] = len(band_bound)
    if band_bound and cfg.max_hits == 0 and cfg.t_min == 0 and cfg.alpha_max >= 1:
        # On the rays with a guard-band decision the GPU's colour is also held against the colour of the oracle's OWN lists,
        # within what those decisions can move it by (the replay below checks the arithmetic on the GPU's lists).
        own, _, _ = v.composite()
        own = own.reshape(-1, 3)
        gcol = gpu["color"].reshape(-1, 3).astype(np.float64)
        for r, b in band_bound.items():
            assert np.all(np.abs(gcol[r] - own[r]) <= b + 1e-4 * np.abs(own[r]) + 1e-6), ("banded ray moved further than its decisions allow", r, gcol[r], own[r], b)
    assert stats["band_hit"] + stats["band_order"] <= max(2, 1e-3 * stats["oracle_hits"])
    # replay the GPU's lists
    v2 = orc.View(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32, bg=cfg.background, max_hits=cfg.max_hits,
                  t_min=cfg.t_min_f32, alpha_max=cfg.alpha_max_f32 if cfg.alpha_max < 1.0 else 1.0, kernel_degree=cfg.kernel_degree)
    v2.set_hits(g_new_off, g_sel_gid)
    color, t_final, cnt = v2.composite()
    stats["margin_t_min"], stats["margin_alpha_max"] = v2.margins()
    grad, gabs, gelem, gterms, gcond = v2.backward(np.asarray(dL_dC, dtype=np.float64), with_abs=True, with_elem=True, with_terms=True,
                                                   with_cond=True)
    return {"color": color, "t_final": t_final, "grad": grad, "gabs": gabs, "gelem": gelem, "gterms": gterms, "gcond": gcond, "stats": stats,
            "sel": sel, "view": v2}


LT32_EPS = 1e-5


def check_lt32(gpu, ref, keep_rays=None):
    """The 16-byte entries the forward wrote, in both layouts, against the oracle's entries of the same hits: the clamp
    flags identical on every composited hit, and every word within LT32_EPS times the oracle's conditioning figure of the
    word (the mass of the two products it is a difference of, plus the effect of a unit relative error of every alpha in
    front of and at the hit: (1 + kappa) |w c| + r ((1 + r) |B| + B_kappa) with r = alpha / (1 - alpha); (1 + kappa) w for
    the weight).  LT32_EPS = 1e-5 covers an alpha evaluated in single precision (a few 1e-6: the exponent is a
    quadratic form of rounded inputs, and where its terms cancel, as for a camera inside a large Gaussian, its absolute error
    of a few 1e-6 is alpha's relative error) plus the roundings of the products and of the sums B and T, and 2e-6 of the word for the (at most four) low mantissa bits that carry the flags and, in the
    primitive-major layout, the pixel index.  Only for a replay of every ray.  Returns the largest error in units of
    the bound."""
    entry, flags, cond = ref["view"].lt_entries(with_cond=True)
    hk = np.ones(entry.shape[0], bool) if keep_rays is None else np.repeat(keep_rays, np.diff(gpu["ray_off"].astype(np.int64)))
    worst = 0.0
    for lt, slots, mask in ((gpu["lt"], gpu["ray_slot"], (~7, ~7, ~7, ~15)), (gpu["tile"]["lt"], gpu["tile"]["ray_slot"], (~0, ~0, ~0, ~7))):
        assert slots.size == entry.shape[0]
        bits = np.ascontiguousarray(lt[slots.astype(np.int64)]).view(np.uint32).reshape(-1, 4)
        f = (bits[:, 3] & 7).astype(np.uint8)
        val = (bits & np.array(mask, np.int64).astype(np.uint32)).view(np.float32).astype(np.float64)
        live = hk & (entry[:, 3] > 0)
        assert np.array_equal(f[live], flags[live])
        tol = LT32_EPS * cond + 2e-6 * np.abs(entry) + 1e-30
        err = np.abs(val - entry)[hk] / tol[hk]
        assert np.all(err <= 1.0), ("LT entry outside its bound", float(err.max()))
        assert np.all(val[hk & (entry[:, 3] == 0)] == 0)           # a hit that is not composited: zero entry
        worst = max(worst, float(err.max(initial=0.0)))
    return worst


def check_lt16(gpu, ref, keep_rays=None):
    """The 8-byte entries the forward wrote (lt_format 2) against the oracle's entries of the same hits: flags
    identical, every colour word within the encoding's 2^-10 and the weight within 2^-11, plus the fp32 error of
    the encoder's input (the colour word is a difference of two products of size about w and alpha/(1-alpha) B).
    Only for a replay of every ray (the oracle's hit order is then the GPU's list order)."""
    import lt16
    entry, flags = ref["view"].lt_entries()
    slots = gpu["tile"]["ray_slot"].astype(np.int64)      # (8-byte entries live in the tile-major layout)
    assert entry.shape[0] == slots.size
    dec, f = lt16.decode(gpu["lt16"][slots])
    if keep_rays is not None:       # (rays left out of the comparison: see the caller)
        hk = np.repeat(keep_rays, np.diff(gpu["ray_off"].astype(np.int64)))
        entry, flags, dec, f = entry[hk], flags[hk], dec[hk], f[hk]
    assert np.array_equal(f, flags)
    x, w = entry[:, :3], entry[:, 3]
    fp32 = 1e-5 * (np.abs(x) + 8.0 * w[:, None])
    assert np.all(np.abs(dec[:, :3] - x) <= 1.02 * lt16.REL_X * np.abs(x) + fp32 + lt16.ABS_SUB)
    assert np.all(np.abs(dec[:, 3] - w) <= 1.02 * lt16.REL_W * w + 1e-5 * w + lt16.ABS_SUB)
    # and the encoding is used to its precision: the typical error is that of nine / ten mantissa bits, not more
    big = np.abs(x) > 1e-6
    assert np.median(np.abs(dec[:, :3] - x)[big] / np.abs(x)[big]) > 2.0 ** -14


def color_errors(gpu, ref, sel, cam):
    c_g = gpu["color"].reshape(-1, 3)[sel].astype(np.float64)
    c_o = ref["color"].reshape(-1, 3)[sel]
    t_g = gpu["t_final"].reshape(-1)[sel].astype(np.float64)
    t_o = ref["t_final"].reshape(-1)[sel]
    return np.abs(c_g - c_o), np.abs(c_o), np.abs(t_g - t_o), np.abs(t_o)


def pack_grad(grad64, K):
    """Oracle layout [n, 11+3K] -> library layout [n, 64]."""
    out = np.zeros((grad64.shape[0], G.GRAD_WORDS))
    out[:, :11 + 3 * K] = grad64
    return out
