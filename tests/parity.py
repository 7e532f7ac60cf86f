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


def run_gpu(scene, cam, cfg: G.Config, dL_dC, cap_pairs=None, cap_hits=None, atomic=True):
    """Full device path for one view; returns numpy copies of every output."""
    g = G.Gaussians.from_numpy(scene)
    if cap_pairs is None or cap_hits is None:
        P, S = G.size_view(cfg, g, cam, slack=1.0)
        cap_pairs = P if cap_pairs is None else cap_pairs
        cap_hits = S if cap_hits is None else cap_hits
    buf = G.ViewBuffers(g.n, g.sh_degree, cam, cfg, cap_pairs, cap_hits)
    dl = torch.from_numpy(np.ascontiguousarray(dL_dC, dtype=np.float32)).cuda()
    G.run_bounds_tile_map(cfg, g, cam, buf)
    G.run_forward(cfg, g, cam, buf)
    G.run_backward(cfg, g, cam, buf, dl)
    counts = G.gart_read_counts(buf.counts)
    out = {"counts": counts, "buf": buf, "g": g, "dl": dl}
    P, H = counts[G.CNT_PAIRS], counts[G.CNT_HITS]
    out["rect"], out["cls"] = to_np(buf.rect)[:g.n], to_np(buf.cls)[:g.n]
    out["tile_off"] = u32(to_np(buf.tile_off))
    if counts[G.CNT_ERROR]:
        return out
    out["pair_gid"] = u32(to_np(buf.pair_gid))[:P]
    out["pair_mask"] = u32(to_np(buf.pair_mask))[:P]
    out["pair_order"] = u32(to_np(buf.pair_order))[:P]
    out["rank_sid"] = u32(to_np(buf.rank_sid))[:P]
    out["slot_of_gid"], out["gid_of_slot"] = u32(to_np(buf.slot_of_gid))[:g.n], u32(to_np(buf.gid_of_slot))[:g.n]
    out["rank_mask"] = u32(to_np(buf.rank_mask))[:P]
    out["rank_gstart"] = u32(to_np(buf.rank_gstart))[:P]
    out["tile_lt_base"] = u32(to_np(buf.tile_lt_base))
    out["color"], out["t_final"] = to_np(buf.color), to_np(buf.t_final)
    out["hit_count"] = u32(to_np(buf.hit_count))
    out["ray_off"] = u32(to_np(buf.ray_off))
    out["ray_gid"] = u32(to_np(buf.ray_gid))[:H]
    out["ray_slot"] = u32(to_np(buf.ray_slot))[:H]
    out["lt"] = to_np(buf.lt)[:counts[G.CNT_LT_SLOTS]]
    out["grad"] = to_np(buf.grad)[:g.n].copy()
    if atomic:
        ga = torch.empty_like(buf.grad)
        G.run_backward_atomic(cfg, g, cam, buf, dl, ga)
        torch.cuda.synchronize()
        out["grad_atomic"] = to_np(ga)[:g.n]
        gw = torch.empty_like(buf.grad)
        G.run_backward_warp(cfg, g, cam, buf, dl, gw)          # ownership ablation: a warp per pair
        torch.cuda.synchronize()
        out["grad_warp"] = to_np(gw)[:g.n]
        import dataclasses
        if cfg.max_hits == 0:   # (the hybrid backward re-derives every alpha in its pixel pass: it takes no hit cap)
            # hybrid backward: the forward again with 4-byte LT entries (same buffers, everything else unchanged)
            cfg_h = dataclasses.replace(cfg, lt_format=1)
            G.run_forward(cfg_h, g, cam, buf)
            gh = torch.empty_like(buf.grad)
            G.run_backward_hybrid(cfg_h, g, cam, buf, dl, gh)
            torch.cuda.synchronize()
            assert G.gart_read_counts(buf.counts)[G.CNT_ERROR] == 0
            out["grad_hybrid"] = to_np(gh)[:g.n]
            # the other outputs of the forward do not depend on the LT format
            assert np.array_equal(to_np(buf.color), out["color"]) and np.array_equal(u32(to_np(buf.ray_gid))[:H], out["ray_gid"])
        # 8-byte LT entries (four halves per hit) and the primitive-centric backward on them
        cfg_8 = dataclasses.replace(cfg, lt_format=2)
        G.run_forward(cfg_8, g, cam, buf)
        g8 = torch.empty_like(buf.grad)
        G.run_backward(cfg_8, g, cam, buf, dl, g8)
        torch.cuda.synchronize()
        assert G.gart_read_counts(buf.counts)[G.CNT_ERROR] == 0
        out["grad_lt16"] = to_np(g8)[:g.n]
        out["lt16"] = to_np(buf.lt).reshape(-1).view(np.uint16)[:4 * counts[G.CNT_LT_SLOTS]].reshape(-1, 4).copy()
        assert np.array_equal(to_np(buf.color), out["color"]) and np.array_equal(u32(to_np(buf.ray_slot))[:H], out["ray_slot"])
    return out


def check_maps(scene, cam, cfg: G.Config, gpu):
    """Rectangles, classes and tile lists against the oracle (bit-exact outside the 1e-9 margin)."""
    osc = orc.OracleScene.from_scene(scene)
    rect, cls, margin = orc.bounds(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32)
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


def check_structure(cam, cfg: G.Config, gpu, max_rays=20000, seed=0):
    """Properties that hold at any size, checked on the whole view without the oracle (the per-hit
    part on a random subset of rays when the view has more than a few million hits)."""
    H = gpu["counts"][G.CNT_HITS]
    L = gpu["counts"][G.CNT_LT_SLOTS]
    ray_off, hit_count = gpu["ray_off"].astype(np.int64), gpu["hit_count"].reshape(-1).astype(np.int64)
    assert ray_off[0] == 0 and ray_off[-1] == H and np.array_equal(np.diff(ray_off), hit_count)
    assert gpu["counts"][G.CNT_MAX_RAY_HITS] == (hit_count.max() if hit_count.size else 0)
    pc = np.bitwise_count(gpu["pair_mask"]).sum(axis=1).astype(np.int64)
    assert pc.sum() == H and L >= H
    # every hit owns exactly one slot
    slots_all = gpu["ray_slot"]
    assert np.unique(slots_all).size == H and (int(slots_all.max()) if H else -1) < L
    ts = cfg.tile_size
    tiles_x = -(-cam.width // ts)
    tile_off, base = gpu["tile_off"].astype(np.int64), gpu["tile_lt_base"].astype(np.int64)
    assert base[0] == 0 and base[-1] == L and np.all(np.diff(base) >= 0)
    n_tile = np.diff(tile_off)
    P = pc.size
    tile_of_pair = np.repeat(np.arange(n_tile.size), n_tile)
    # pair_order: a permutation of each tile's pairs in descending hit count, stable
    order = gpu["pair_order"].astype(np.int64)
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
    assert np.array_equal(gpu["rank_sid"], gpu["slot_of_gid"][gpu["pair_gid"][order]])
    assert np.array_equal(gpu["rank_mask"], gpu["pair_mask"][order])
    # slots: visible Gaussians in the order of the tile row of their rectangle's corner, ids ascending inside a row
    rect_ = gpu["rect"]
    vis = rect_[:, 2] >= rect_[:, 0]
    V = int(vis.sum())
    key_ = rect_[:, 1] // ts
    want_order = np.nonzero(vis)[0][np.argsort(key_[vis], kind="stable")]
    assert np.array_equal(gpu["gid_of_slot"][:V], want_order.astype(np.uint32)) and np.all(gpu["gid_of_slot"][V:] == 0xffffffff)
    inv = np.full(rect_.shape[0], 0xffffffff, np.uint32)
    inv[want_order] = np.arange(V, dtype=np.uint32)
    assert np.array_equal(gpu["slot_of_gid"], inv)
    # rank_gstart: start of the 32-rank group; a group spans 32 x its largest (= first) count
    gs_ = gpu["rank_gstart"].astype(np.int64)                   # by position in rank order
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
    # ---- per hit: on all rays, or on a random subset of them
    n_rays = hit_count.size
    if H > 5_000_000:
        rsel = np.sort(np.random.default_rng(seed).choice(n_rays, size=max_rays, replace=False))
    else:
        rsel = np.arange(n_rays)
    cnt = hit_count[rsel]
    idx = np.repeat(ray_off[rsel], cnt) + (np.arange(cnt.sum()) - np.repeat(np.cumsum(cnt) - cnt, cnt))
    rays = np.repeat(rsel, cnt)
    slots = gpu["ray_slot"][idx].astype(np.int64)
    gids = gpu["ray_gid"][idx].astype(np.int64)
    tile = (rays // cam.width) // ts * tiles_x + (rays % cam.width) // ts
    rel = slots - base[tile]
    assert np.all(rel >= 0) and np.all(slots < base[tile + 1])
    # locate the pair: among the tile's pairs, the one whose Gaussian is the hit's (ids ascend in a tile)
    pair_gid = gpu["pair_gid"].astype(np.int64)
    mul = int(pair_gid.max()) + 1 if P else 1
    key = tile_of_pair * mul + pair_gid
    want = tile * mul + gids
    pair = np.searchsorted(key, want)
    assert np.array_equal(key[pair], want)
    e = rel - slot0[pair]
    assert np.all(e % 32 == 0) and np.all(e >= 0) and np.all(e // 32 < pc[pair])
    # the e-th hit of a pair is its e-th set mask bit in pixel order
    px = (rays % cam.width) % ts + ((rays // cam.width) % ts) * ts
    words = gpu["pair_mask"][pair]                                  # [h, MW]
    w_idx, b_idx = px // 32, px % 32
    word = words[np.arange(pair.size), w_idx].astype(np.uint64)
    assert np.all((word >> b_idx.astype(np.uint64)) & np.uint64(1))
    below = np.bitwise_count(word & ((np.uint64(1) << b_idx.astype(np.uint64)) - np.uint64(1))).astype(np.int64)
    for q in range(words.shape[1]):
        below += np.where(q < w_idx, np.bitwise_count(words[:, q]).astype(np.int64), 0)
    assert np.array_equal(below, e // 32)
    # LT: word 3 is the blending weight T alpha in (0, 1) with the three clamp flags in its low mantissa
    # bits; the vector part is finite.  (The values themselves are checked through the gradients.)
    used = gpu["lt"][slots]
    wgt = (np.ascontiguousarray(used[:, 3]).view(np.uint32) & np.uint32(0xFFFFFFF8)).view(np.float32)
    assert np.all(np.isfinite(used)) and np.all(wgt >= 0) and np.all(wgt < 1.0)
    assert np.all(np.isfinite(gpu["color"])) and np.all(np.isfinite(gpu["grad"]))


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
    v = orc.View(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32, bg=cfg.background)
    v.find_hits(mode, pixel_mask)
    o_off, o_gid, o_t, o_alpha = v.hits()
    g_off, g_gid = gpu["ray_off"].astype(np.int64), gpu["ray_gid"]
    o_off = o_off.astype(np.int64)
    stats = {"rays": int(sel.size), "oracle_hits": int(o_off[-1]), "band_hit": 0, "band_order": 0}
    g_cnt, o_cnt = g_off[sel + 1] - g_off[sel], o_off[sel + 1] - o_off[sel]
    # fast path: concatenate selected lists and compare wholesale
    g_new_off, g_sel_gid = _lists_for(gpu["ray_off"].astype(np.int64), g_gid, sel)
    identical = np.array_equal(g_cnt, o_cnt) and np.array_equal(g_sel_gid, o_gid)
    if not identical:
        amin = cfg.alpha_min_f32
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
    stats["identical_lists"] = bool(identical)
    assert stats["band_hit"] + stats["band_order"] <= max(2, 1e-3 * stats["oracle_hits"])
    # replay the GPU's lists
    v2 = orc.View(osc, cam, alpha_min=cfg.alpha_min_f32, near=cfg.near_f32, bg=cfg.background, max_hits=cfg.max_hits)
    v2.set_hits(g_new_off, g_sel_gid)
    color, t_final, cnt = v2.composite()
    grad, gabs, gelem, gterms = v2.backward(np.asarray(dL_dC, dtype=np.float64), with_abs=True, with_elem=True, with_terms=True)
    return {"color": color, "t_final": t_final, "grad": grad, "gabs": gabs, "gelem": gelem, "gterms": gterms, "stats": stats,
            "sel": sel, "view": v2}


def check_lt16(gpu, ref):
    """The 8-byte entries the forward wrote (lt_format 2) against the oracle's entries of the same hits: flags
    identical, every colour word within the encoding's 2^-10 and the weight within 2^-11, plus the fp32 error of
    the encoder's input (the colour word is a difference of two products of size about w and alpha/(1-alpha) B).
    Only for a replay of every ray (the oracle's hit order is then the GPU's list order)."""
    import lt16
    entry, flags = ref["view"].lt_entries()
    slots = gpu["ray_slot"].astype(np.int64)
    assert entry.shape[0] == slots.size
    dec, f = lt16.decode(gpu["lt16"][slots])
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
