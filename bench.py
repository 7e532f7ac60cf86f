"""Benchmark of the gart hot path on B200: one step = bounds -> tile map -> forward -> backward of one view.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config unbounded6m] [--tile-size 8]
    python bench.py --impl reference ...      # the float64 CPU oracle on the host cores, bounded sample

Prints ONE JSON line.  `value` is ray-Gaussian hits per second over the whole step with every input
resident in HBM; `e2e` is the same metric through the host-buffer entry point (gart_view_host) with
the host<->device copies inside the timed region.  Per-stage times, the backward's roofline
fraction, the speedup over the pixel-centric atomic backward, clocks sampled during the timed region
and the oracle timed on the host cores are reported in the same line.

With N > 1 (torchrun) the views of the orbit are sharded over the ranks; ranks exchange nothing on
the data path (views are independent), so the scaling is "weak".
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gart_scenes as gs  # noqa: E402

METRIC = "ray_gaussian_hits_per_s"
UNIT = "hits/s"
HBM_FALLBACK_GBS = 6650.0


# ----------------------------------------------------------------------------------------- host logic
def shard_views(n_views: int, rank: int, world: int):
    """Views handled by `rank`: round-robin, every rank gets at least one (wrapping if world > n_views)."""
    mine = [v for v in range(n_views) if v % world == rank]
    return mine if mine else [rank % n_views]


def _radix_passes(n_keys: int) -> int:
    bits = 1
    while (1 << bits) <= n_keys:          # keys 0 .. n_keys (the last one marks "none")
        bits += 1
    return (bits + 7) // 8


def launches_per_step(width: int, height: int, tile_size: int, layout: str = "tile") -> int:
    """Kernel launches of one step (memsets are not kernels).  A scan is three kernels, a radix pass histogram + scan +
    scatter."""
    tiles = -(-width // tile_size) * -(-height // tile_size)
    sups_x, sups_y = -(-width // 16), -(-height // 16)           # super-tiles of 16 x 16 pixels
    scan, radix = 3, 5
    tile_map = 1 + scan + 1 + 1 + _radix_passes(tiles - 1) * radix + 1   # areas, scan, total, emission, pair sort, offsets
    if layout == "tile":
        bounds = 1 + _radix_passes(sups_y) * radix + 1           # bounds kernel, slot sort on the corner's super-tile row, record gather
        forward = 1 + 1 + scan + scan + 1 + 1 + 2                # mask, tile sort, entries per tile, ray offsets, totals, evaluation, sweep per ray-length class
        backward = 4                                             # zero, pair kernel, per-slot conversion, scatter of the SH gradient
        return bounds + tile_map + forward + backward
    sups = sups_x * sups_y
    bounds = 1 + _radix_passes(sups) * radix + 1                 # ... slot sort on the corner's super-tile
    forward = (scan + 1 + 1 + scan                               # pairs per slot, mask, tile sort, entries per tile
               + scan + 1 + 1 + _radix_passes(sups - 1) * radix  # items per slot, total, emission, item sort on the super-tile
               + 1 + 1 + 1 + scan + scan + 1 + 1 + 1             # segment offsets, descriptors, ranking, two scans, blocks, LT bases, per-rank copy
               + scan + 1 + 1 + 2)                               # ray offsets, totals, evaluation, sweep per ray-length class
    backward = 4                                                 # records of cut Gaussians zeroed, zero rows, item kernel, conversion of cut Gaussians
    return bounds + tile_map + forward + backward


def algorithmic_bytes_backward(H, P, n_vis, n_pixels, K):
    """Bytes the primitive-centric backward must move once per view: the LT entry of every hit (16 B), the pair
    list (4 B per pair), each visible Gaussian's parameters and SH read once (13 + 3K words), its gradient written
    once (11 + 3K words), and per pixel dL/dC, C and T_final (28 B)."""
    return 16 * H + 4 * P + 4 * (13 + 3 * K) * n_vis + 4 * (11 + 3 * K) * n_vis + 28 * n_pixels


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the kernels of gart_backward, from the ncu captures
# summarised in profiles/dram_traffic_unbounded6m_crop.md (8x8 tiles, SH degree 3, central crop of a view), each
# divided by the unit it grows with.  Tile-major layout: the pair kernel by hits, zeroing and conversion by visible
# Gaussians, the scatter's reads by visible Gaussians and its writes by all Gaussians.  Primitive-major layout: the item
# kernel's reads by LT entries (it streams the padded buffer) and its writes by visible Gaussians, the zero rows by the
# Gaussians without a slot, the two kernels for cut Gaussians by visible Gaussians.  `--crop 0.5` prints the units of the captured case in roofline.traffic_units, so
# that a fresh capture divides into these figures.
TRAFFIC_MODEL = {
    "tile": {"pairs_per_hit": 39.9, "zero_per_visible": 214.6, "convert_per_visible": 153.3,
             "scatter_read_per_visible": 186.0, "scatter_write_per_gaussian": 220.7},
    "primitive": {"items_read_per_lt_entry": 21.91, "items_write_per_visible": 235.7, "fill_write_per_invisible": 238.6,
                  "fill_read_per_gaussian": 4.0, "big_per_visible": 38.8},
}


def measured_traffic_backward(layout, H, L, n_vis, n):
    t = TRAFFIC_MODEL[layout]
    if layout == "tile":
        return (t["pairs_per_hit"] * H + (t["zero_per_visible"] + t["convert_per_visible"] + t["scatter_read_per_visible"]) * n_vis
                + t["scatter_write_per_gaussian"] * n)
    return (t["items_read_per_lt_entry"] * L + (t["items_write_per_visible"] + t["big_per_visible"]) * n_vis
            + t["fill_write_per_invisible"] * (n - n_vis) + t["fill_read_per_gaussian"] * n)


def fp32_instr_backward(H, K):
    """FP32-pipe instructions per hit of the backward: evaluation 31, maximum-response point 9, colour and
    SH gradient 2*3K, alpha gradient 14, moments 13."""
    return H * (31 + 9 + 6 * K + 14 + 13)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured", float(d.get("sm_max_mhz", 1965.0))
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback", 1965.0


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = "clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
            "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + q, "--format=csv,noheader,nounits",
                                          "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nme, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------- workload
def make_workload(name: str, n_views=None, crop=1.0):
    """Scene and cameras of a configuration.  crop < 1 keeps the central part of every image (same
    focal length, fewer pixels): a smaller case of the same per-tile structure, used for profiling."""
    kw = {}
    if n_views is not None and name in ("shell200k", "unbounded1m", "unbounded6m"):
        kw["n_views"] = n_views
    scene, cams = gs.make(name, **kw)
    if crop < 1.0:
        cams = [gs.Camera(max(8, int(c.width * crop)), max(8, int(c.height * crop)), c.fx, c.fy,
                          max(8, int(c.width * crop)) / 2.0, max(8, int(c.height * crop)) / 2.0, c.w2c) for c in cams]
    return scene, cams


def oracle_sample(scene, cam, seed=0, frac=0.02, tile=8):
    """Pixel mask for the oracle's bounded sample: a random subset of 8x8 tiles of the view."""
    rng = np.random.default_rng([seed, 0x51])
    tx, ty = -(-cam.width // tile), -(-cam.height // tile)
    pick = rng.random((ty, tx)) < frac
    mask = np.repeat(np.repeat(pick, tile, axis=0), tile, axis=1)[:cam.height, :cam.width]
    return np.ascontiguousarray(mask.astype(np.uint8))


def time_oracle(scene, cam, dL_dC, frac, threads=None, split=False):
    """Oracle (as it stands) on a bounded sample of the view (frac >= 1: every ray): hit discovery + ordering +
    compositing + backward for the sampled rays.  Returns (hits, seconds, threads, rays); with split=True the seconds are
    (forward, backward)."""
    from oracle import gart_oracle as orc
    all_threads = orc.max_threads()
    if threads:
        orc.set_threads(threads)
    osc = orc.OracleScene.from_scene(scene)
    mask = oracle_sample(scene, cam, frac=frac) if frac < 1.0 else None
    t0 = time.perf_counter()
    v = orc.View(osc, cam, alpha_min=float(np.float32(1.0 / 255.0)), near=float(np.float32(0.01)))
    H = v.find_hits(orc.PREFILTER, mask)
    v.composite()
    t1 = time.perf_counter()
    v.backward(np.asarray(dL_dC, dtype=np.float64))
    t2 = time.perf_counter()
    v.close()
    used = orc.max_threads()
    if threads:
        orc.set_threads(all_threads)
    rays = int(mask.sum()) if mask is not None else cam.width * cam.height
    return H, ((t1 - t0, t2 - t1) if split else t2 - t0), used, rays


def oracle_detail(config="cluster10k"):
    """The oracle on every ray of one view of a small configuration, forward (hit discovery, ordering, compositing) and
    backward timed separately, with all host threads and with one."""
    scene, cams = gs.make(config)
    cam = cams[0]
    g = gs.upstream_gradient(cam, 0)
    out = {"workload": config, "unit": UNIT}
    for key, thr in (("all_threads", None), ("one_thread", 1)):
        H, (tf, tb), used, rays = time_oracle(scene, cam, g, 1.0, threads=thr, split=True)
        out[key] = {"cores": used, "hits": H, "forward_s": tf, "backward_s": tb, "value": H / (tf + tb),
                    "forward_hits_per_s": H / tf, "backward_hits_per_s": H / tb}
    return out


def run_reference(args):
    """--impl reference: the oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    scene, cams = make_workload(args.config, crop=args.crop)
    frac = args.oracle_frac / 4.0     # per step; keeps a K-step run within minutes
    times, hits = [], 0
    for s in range(args.warmup + args.steps):
        cam = cams[s % len(cams)]
        g = gs.upstream_gradient(cam, s % len(cams))
        H, dt, thr, npx = time_oracle(scene, cam, g, frac)
        if s >= args.warmup:
            times.append(dt); hits += H
    total = sum(times)
    val = hits / total if total > 0 else 0.0
    sample = "random %.2f%% of the 8x8 tiles of each view (%d rays), all Gaussians, one view per step" % (100 * frac, npx)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.config, "n_gaussians": scene.n, "width": cams[0].width, "height": cams[0].height,
                       "sh_degree": scene.sh_degree, "tile_size": args.tile_size, "views": len(cams), "crop": args.crop},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------- GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2608_17298_b200.gart as G

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the gart library")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    tile_major = args.lt_layout == "tile"
    cfg = G.Config(tile_size=args.tile_size, lt_layout=G.LT_TILE_MAJOR if tile_major else G.LT_PRIMITIVE_MAJOR)
    run_backward = G.run_backward_tile if tile_major else G.run_backward
    scene, cams = make_workload(args.config, crop=args.crop)
    mine = shard_views(len(cams), rank, world)
    g = G.Gaussians.from_numpy(scene, dev)
    K = (scene.sh_degree + 1) ** 2
    dls = {v: torch.from_numpy(gs.upstream_gradient(cams[v], v)).to(dev) for v in mine}

    # capacities: exact pair count and slot bound of this rank's first view, with slack for the other views
    cap_pairs, cap_hits = G.size_view(cfg, g, cams[mine[0]], slack=args.slack, device=dev)
    buf = G.ViewBuffers(g.n, g.sh_degree, cams[0], cfg, cap_pairs, cap_hits, dev)
    stream = torch.cuda.current_stream()

    def step(v, ev=None):
        cam = cams[v]
        if ev: ev[0].record(stream)
        G.run_bounds_tile_map(cfg, g, cam, buf, stream)
        if ev: ev[1].record(stream)
        G.run_forward(cfg, g, cam, buf, stream, ray_lists=False)   # the ordered per-ray lists serve only the atomic baseline
        if ev: ev[2].record(stream)
        run_backward(cfg, g, cam, buf, dls[v], None, stream)
        if ev: ev[3].record(stream)

    for s in range(args.warmup):
        step(mine[s % len(mine)])
    torch.cuda.synchronize()
    cnt = G.gart_read_counts(buf.counts)
    if cnt[G.CNT_ERROR]:
        raise RuntimeError("capacity exceeded during warm-up: counts=%s cap_pairs=%d cap_hits=%d" % (cnt, cap_pairs, cap_hits))

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    hits_ev = []
    sampler = ClockSampler(local)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    counts_log = torch.zeros((args.steps, G.COUNTS_WORDS), dtype=torch.int32, device=dev)
    t_start.record(stream)
    for s in range(args.steps):
        step(mine[s % len(mine)], evs[s])
        counts_log[s].copy_(buf.counts)          # device-to-device, 32 bytes: keeps per-view counts without a host sync
    t_end.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    total_ms = t_start.elapsed_time(t_end)
    cl = counts_log.cpu().numpy().view(np.uint32).astype(np.int64)
    if (cl[:, G.CNT_ERROR] != 0).any():
        raise RuntimeError("capacity exceeded inside the timed region: %s" % cl.tolist())
    hits_total = int(cl[:, G.CNT_HITS].sum())
    stage = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in evs])   # maps, forward, backward
    bwd_ms = float(np.mean(stage[:, 2]))

    # whole-job aggregate: total hits of all ranks / max time over ranks
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        h = torch.tensor([hits_total], dtype=torch.float64, device=dev)
        dist.all_reduce(h, op=dist.ReduceOp.SUM)
        total_ms_all, hits_all = float(t.item()), float(h.item())
    else:
        total_ms_all, hits_all = total_ms, float(hits_total)

    # ---- the other backward passes, each on the last view's buffers
    import dataclasses
    last_v = mine[(args.steps - 1) % len(mine)]
    ga = torch.empty_like(buf.grad)

    def timed(fn, reps):
        ts_ = []
        for i in range(reps + 1):                                # one untimed run first
            a0 = torch.cuda.Event(enable_timing=True); a1 = torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            fn()
            a1.record(stream)
            torch.cuda.synchronize()
            if i > 0:
                ts_.append(a0.elapsed_time(a1))
        return float(np.mean(ts_))

    # pixel-centric baselines (Sec. 3.5): one atomicAdd per gradient word per hit, and the same sums as 16-byte vector reductions
    atomic_ms, atomic_vec_ms = None, None
    if args.atomic_reps > 0:
        G.run_forward(cfg, g, cams[last_v], buf, stream, ray_lists=True)   # same view again, this time with the lists
        atomic_ms = timed(lambda: G.run_backward_atomic(cfg, g, cams[last_v], buf, dls[last_v], ga, stream), args.atomic_reps)
        cfg_v = dataclasses.replace(cfg, atomic_mode=1)
        atomic_vec_ms = timed(lambda: G.run_backward_atomic(cfg_v, g, cams[last_v], buf, dls[last_v], ga, stream), args.atomic_reps)
    # the other layout of the intermediate buffer and the backward pass that reads it (primitive-major: a thread walks all
    # hits of a Gaussian and writes its gradient record once; tile-major: the paper's block per tile with one vector atomic
    # update per pair), bounds to backward of the same view in buffers of its own (the slot order follows the layout)
    other_layout = None
    if args.layout_reps > 0:
        cfg_a = dataclasses.replace(cfg, lt_layout=G.LT_PRIMITIVE_MAJOR if tile_major else G.LT_TILE_MAJOR)
        pa, ha = G.size_view(cfg_a, g, cams[last_v], slack=1.0, device=dev)
        ba = G.ViewBuffers(g.n, g.sh_degree, cams[last_v], cfg_a, pa, ha, dev)
        other_layout = {"layout": "primitive" if tile_major else "tile",
                        "bounds_tile_map": timed(lambda: G.run_bounds_tile_map(cfg_a, g, cams[last_v], ba, stream), args.layout_reps),
                        "forward": timed(lambda: G.run_forward(cfg_a, g, cams[last_v], ba, stream, ray_lists=False), args.layout_reps),
                        "backward": timed(lambda: G.run_backward(cfg_a, g, cams[last_v], ba, dls[last_v], None, stream), args.layout_reps)}
        ca = G.gart_read_counts(ba.counts)
        if ca[G.CNT_ERROR]:
            raise RuntimeError("capacity exceeded in the other layout: %s" % ca)
        other_layout["lt_entries"] = int(ca[G.CNT_LT_SLOTS])
        del ba
        torch.cuda.empty_cache()
    # the ownership ablation (a warp per pair instead of a thread), tile-major layout
    cfg_t = dataclasses.replace(cfg, lt_layout=G.LT_TILE_MAJOR)
    warp_ms = None
    if args.warp_reps > 0:
        G.run_forward(cfg_t, g, cams[last_v], buf, stream, ray_lists=False)
        warp_ms = timed(lambda: G.run_backward_warp(cfg_t, g, cams[last_v], buf, dls[last_v], ga, stream), args.warp_reps)
    # hybrid backward (colour gradients primitive-centric from 4 bytes per hit, the rest pixel-centric), same view
    hybrid_ms = None
    if args.hybrid_reps > 0:
        cfg_h = dataclasses.replace(cfg, lt_format=1, lt_layout=G.LT_TILE_MAJOR)
        G.run_forward(cfg_h, g, cams[last_v], buf, stream, ray_lists=True)
        hybrid_ms = timed(lambda: G.run_backward_hybrid(cfg_h, g, cams[last_v], buf, dls[last_v], ga, stream), args.hybrid_reps)
    # 8-byte LT entries (four halves per hit): forward and block-per-tile backward of the same view
    lt16_ms = None
    if args.lt16_reps > 0:
        cfg_8 = dataclasses.replace(cfg, lt_format=2, lt_layout=G.LT_TILE_MAJOR)
        f8 = timed(lambda: G.run_forward(cfg_8, g, cams[last_v], buf, stream, ray_lists=False), args.lt16_reps)
        b8 = timed(lambda: G.run_backward_tile(cfg_8, g, cams[last_v], buf, dls[last_v], ga, stream), args.lt16_reps)
        lt16_ms = {"forward": f8, "backward": b8}
    # the other tile size: the whole step of the same view in buffers of its own
    other_ts = None
    if args.other_ts_reps > 0:
        cfg_o = dataclasses.replace(cfg, tile_size=16 if cfg.tile_size == 8 else 8)
        po, ho = G.size_view(cfg_o, g, cams[last_v], slack=1.0, device=dev)
        bo = G.ViewBuffers(g.n, g.sh_degree, cams[last_v], cfg_o, po, ho, dev)
        other_ts = {"tile_size": cfg_o.tile_size,
                    "bounds_tile_map": timed(lambda: G.run_bounds_tile_map(cfg_o, g, cams[last_v], bo, stream), args.other_ts_reps),
                    "forward": timed(lambda: G.run_forward(cfg_o, g, cams[last_v], bo, stream, ray_lists=False), args.other_ts_reps),
                    "backward": timed(lambda: G.run_backward(cfg_o, g, cams[last_v], bo, dls[last_v], None, stream), args.other_ts_reps)}
        co = G.gart_read_counts(bo.counts)
        if co[G.CNT_ERROR]:
            raise RuntimeError("capacity exceeded at the other tile size: %s" % co)
        other_ts["pairs"] = int(co[G.CNT_PAIRS])
        del bo
        torch.cuda.empty_cache()
    last = cl[-1]
    prim_last_ms = float(stage[-1, 2])
    del ga

    # ---- end to end through the host-buffer entry point
    e2e = None
    if args.e2e_steps > 0:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()

        class HS:
            pass
        hs = HS()
        hs.mean, hs.scale, hs.quat, hs.opacity, hs.sh = pin(scene.mean), pin(scene.scale), pin(scene.quat), pin(scene.opacity), pin(scene.sh)
        hs.sh_degree = scene.sh_degree
        hdl = {v: pin(gs.upstream_gradient(cams[v], v)) for v in mine}
        cam0 = cams[0]
        color_h = torch.empty((cam0.height, cam0.width, 3), dtype=torch.float32).pin_memory()
        grad_h = torch.empty((scene.n, G.GRAD_WORDS), dtype=torch.float32).pin_memory()
        # free the resident buffers first: the arena holds its own copy of everything
        del buf
        torch.cuda.empty_cache()
        arena_bytes = G.gart_view_host_arena_bytes(scene.n, scene.sh_degree, cam0.width, cam0.height, cfg.tile_size, cap_pairs, cap_hits)
        h2d = 4 * scene.n * (3 + 3 + 4 + 1 + 3 * K) + 12 * cam0.width * cam0.height
        d2h = 4 * scene.n * G.GRAD_WORDS + 12 * cam0.width * cam0.height + 4 * G.COUNTS_WORDS

        def reduce_e2e(hits, secs):
            if world > 1:
                tt = torch.tensor([secs], dtype=torch.float64, device=dev); dist.all_reduce(tt, op=dist.ReduceOp.MAX)
                hh = torch.tensor([hits], dtype=torch.float64, device=dev); dist.all_reduce(hh, op=dist.ReduceOp.SUM)
                return float(hh.item()) / float(tt.item())
            return hits / secs

        # (a) one view at a time: gart_view_host returns when the view's results are on the host
        arena = torch.empty(arena_bytes, dtype=torch.uint8, device=dev)
        e_hits, e_t = 0, 0.0
        for s in range(args.e2e_steps + 1):
            v = mine[s % len(mine)]
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            c = G.gart_view_host(cfg, hs, cams[v], hdl[v], color_h, grad_h, cap_pairs, cap_hits, arena, stream)
            dt = time.perf_counter() - t0
            if s > 0:
                e_hits += c[G.CNT_HITS]; e_t += dt
        serial = {"value": reduce_e2e(e_hits, e_t), "ms_per_step": 1e3 * e_t / args.e2e_steps}
        # (b) several views in flight (gart_view_host_async on one stream each, with an arena and host arrays of its own): one
        # view's uploads overlap another's downloads and kernels.  Same bytes per step, every copy inside the timed region.
        NS = args.e2e_inflight
        slots = [{"arena": arena, "color": color_h, "grad": grad_h, "stream": torch.cuda.Stream(dev)}]
        for _ in range(NS - 1):
            slots.append({"arena": torch.empty(arena_bytes, dtype=torch.uint8, device=dev),
                          "color": torch.empty_like(color_h).pin_memory(), "grad": torch.empty_like(grad_h).pin_memory(),
                          "stream": torch.cuda.Stream(dev)})
        for sl in slots:
            sl["counts"] = torch.zeros(G.COUNTS_WORDS, dtype=torch.int32).pin_memory()
            sl["busy"] = False
        p_hits = 0

        def drain(sl):
            if sl["busy"]:
                sl["stream"].synchronize()
                st = G.gart_counts_status(sl["counts"])
                if st != G.GART_OK:
                    raise RuntimeError("gart_view_host_async: status %d" % st)
                sl["busy"] = False
                return int(sl["counts"].numpy().view(np.uint32)[G.CNT_HITS])
            return 0

        n_pipe = NS * args.e2e_steps
        for s in range(NS + n_pipe):                    # one untimed view per slot first
            if s == NS:
                for sl in slots:
                    drain(sl)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            sl = slots[s % NS]
            got = drain(sl)                             # the slot's previous view has landed on the host: its arrays are free again
            if s >= 2 * NS:
                p_hits += got
            v = mine[s % len(mine)]
            G.gart_view_host_async(cfg, hs, cams[v], hdl[v], sl["color"], sl["grad"], cap_pairs, cap_hits, sl["counts"], sl["arena"], sl["stream"])
            sl["busy"] = True
        for sl in slots:
            p_hits += drain(sl)
        p_t = time.perf_counter() - t0
        e2e = {"value": reduce_e2e(p_hits, p_t), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": 1e3 * p_t / n_pipe, "steps": n_pipe, "mode": "%d views in flight (gart_view_host_async, one stream each)" % NS,
               "one_view_at_a_time": serial}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant call (gart_backward: zeroing + pair kernel + per-Gaussian conversion)
    hbm, hbm_src, sm_max = measured_peaks()
    n_pix = cams[0].width * cams[0].height
    Hm, Pm, Nv = float(np.mean(cl[:, G.CNT_HITS])), float(np.mean(cl[:, G.CNT_PAIRS])), float(np.mean(cl[:, G.CNT_VISIBLE]))
    Lm = float(np.mean(cl[:, G.CNT_LT_SLOTS]))
    B = algorithmic_bytes_backward(Hm, Pm, Nv, n_pix, K)
    achieved = B / (bwd_ms * 1e-3) / 1e9
    F = fp32_instr_backward(Hm, K)
    alu_peak = 148 * 128 * sm_max * 1e6            # FP32 lane-instructions per second at the maximum SM clock
    roof = {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm, "traffic": None,
            "peak_source": hbm_src,
            "kernel": ("gart_backward, tile-major (bwd_zero + bwd_pairs + bwd_convert + bwd_scatter kernels)" if tile_major else
                       "gart_backward, primitive-major (bwd_gm item kernel + gm_fill zero rows + gm_zero_big / gm_convert_big for cut Gaussians)"),
            "algorithmic_bytes": B, "ms": bwd_ms,
            "alu": {"fp32_lane_instr": F, "peak_lane_instr_per_s": alu_peak, "frac": F / (bwd_ms * 1e-3) / alu_peak}}
    if cfg.tile_size == 8 and scene.sh_degree == 3:
        # captured on a cropped view of unbounded6m and scaled by the units each kernel's traffic grows with
        roof["traffic"] = measured_traffic_backward(args.lt_layout, Hm, Lm, Nv, scene.n)
        roof["traffic_source"] = "ncu capture of a cropped view, scaled (profiles/dram_traffic_unbounded6m_crop.md)"
    roof["traffic_units"] = {"hits": Hm, "lt_entries": Lm, "visible": Nv, "gaussians": scene.n, "model": TRAFFIC_MODEL[args.lt_layout]}

    # ---- the oracle on the host cores, bounded sample (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cam = cams[mine[0]]
        H, dt, thr, npx = time_oracle(scene, cam, gs.upstream_gradient(cam, mine[0]), args.oracle_frac)
        cpu = {"value": H / dt, "unit": UNIT, "cores": thr, "kind": "oracle",
               "sample": "random %.1f%% of the 8x8 tiles of view %d (%d rays, %d hits), all Gaussians, %.1f s" % (
                   100 * args.oracle_frac, mine[0], npx, H, dt),
               "small_config": oracle_detail()}

    line = {
        "metric": METRIC, "value": hits_all / (total_ms_all * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms_all / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.config, "n_gaussians": scene.n, "width": cams[0].width, "height": cams[0].height,
                   "sh_degree": scene.sh_degree, "tile_size": cfg.tile_size, "lt_layout": args.lt_layout, "views": len(cams), "crop": args.crop,
                   "l2": "inputs larger than L2 (parameters %.2f GB, LT %.2f GB per view)" % (
                       4e-9 * scene.n * (11 + 3 * K), 16e-9 * Hm),
                   "hits_per_view": Hm, "pairs_per_view": Pm, "visible_per_view": Nv,
                   "lt_entries_per_view": float(np.mean(cl[:, G.CNT_LT_SLOTS]))},
        "stages_ms": {"bounds_tile_map": float(np.mean(stage[:, 0])), "forward": float(np.mean(stage[:, 1])),
                      "backward": bwd_ms, "backward_median": float(np.median(stage[:, 2]))},
        "backward_hits_per_s": Hm / (bwd_ms * 1e-3),
        "backward_atomic_ms": atomic_ms, "backward_atomic_vector_ms": atomic_vec_ms,
        "speedup_vs_atomic": (atomic_ms / prim_last_ms) if atomic_ms else None,                 # scalar atomicAdd per word (Sec. 3.5)
        "speedup_vs_atomic_vector": (atomic_vec_ms / prim_last_ms) if atomic_vec_ms else None,  # the same sums as 16-byte reductions
        "backward_hybrid_ms": hybrid_ms,
        "lt_8byte_ms": lt16_ms,
        "backward_warp_per_pair_ms": warp_ms,
        "other_layout_ms": other_layout,
        "other_tile_size_ms": other_ts,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step(cams[0].width, cams[0].height, cfg.tile_size, args.lt_layout) * args.steps,
        "roofline": roof, "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="unbounded6m", choices=list(gs.CONFIGS))
    ap.add_argument("--tile-size", type=int, default=8, choices=[8, 16])
    ap.add_argument("--lt-layout", default="tile", choices=["primitive", "tile"],
                    help="layout of the intermediate buffer and the backward pass that reads it: primitive-major (gart_backward) or tile-major (gart_backward_tile)")
    ap.add_argument("--slack", type=float, default=1.25)
    ap.add_argument("--atomic-reps", type=int, default=2)
    ap.add_argument("--warp-reps", type=int, default=1, help="timed runs of the warp-per-pair backward on the last view (0: skip)")
    ap.add_argument("--layout-reps", type=int, default=2, help="timed runs of the whole step in the other layout on the last view (0: skip)")
    ap.add_argument("--hybrid-reps", type=int, default=1, help="timed runs of the hybrid backward on the last view (0: skip)")
    ap.add_argument("--lt16-reps", type=int, default=2, help="timed runs of forward + backward with 8-byte LT entries on the last view (0: skip)")
    ap.add_argument("--other-ts-reps", type=int, default=2, help="timed runs of the whole step at the other tile size on the last view (0: skip)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-inflight", type=int, default=4, help="views in flight in the end-to-end measurement (each holds an arena on the device)")
    ap.add_argument("--oracle-frac", type=float, default=0.08)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--crop", type=float, default=1.0, help="central crop of every view (profiling on a smaller case)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
