"""Host logic of the benchmark: view sharding, launch counting, byte accounting, and the
max-over-ranks / sum-over-ranks aggregation on two gloo ranks (CPU)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def test_shard_views_partition():
    for world in (1, 2, 3, 4, 8, 16, 32):
        seen = []
        for r in range(world):
            mine = bench.shard_views(16, r, world)
            assert len(mine) >= 1
            seen += mine
        if world <= 16:
            assert sorted(seen) == list(range(16))


def test_launch_count_and_bytes():
    # 155 x 103 tiles of 8 pixels (14 key bits: two radix passes of five kernels), 78 x 52 super-tiles (12 bits: two passes)
    assert bench.launches_per_step(1240, 824, 8, "primitive") == (1 + 10 + 1) + (7 + 10) + (8 + (5 + 10) + 12 + 7) + 4
    # 8 x 8 tiles, 4 x 4 super-tiles: one pass each
    assert bench.launches_per_step(64, 64, 8, "primitive") == (1 + 5 + 1) + (7 + 5) + (8 + (5 + 5) + 12 + 7) + 4
    # tile-major layout: the slot sort has 52 super-tile rows (one pass), the forward no item lists
    assert bench.launches_per_step(1240, 824, 8, "tile") == (1 + 5 + 1) + (7 + 10) + 12 + 4
    assert bench.launches_per_step(1240, 824, 8) == bench.launches_per_step(1240, 824, 8, "tile")
    B = bench.algorithmic_bytes_backward(H=100, P=10, n_vis=5, n_pixels=64, K=16)
    assert B == 1600 + 40 + 4 * 61 * 5 + 4 * 59 * 5 + 28 * 64
    # the traffic model adds its per-unit figures
    t = bench.TRAFFIC_MODEL
    tp = t["primitive"]
    assert bench.measured_traffic_backward("primitive", 0, 0, 0, 10) == 10 * (tp["fill_write_per_invisible"] + tp["fill_read_per_gaussian"])
    assert bench.measured_traffic_backward("primitive", 5, 7, 0, 0) == 7 * tp["items_read_per_lt_entry"]
    assert bench.measured_traffic_backward("primitive", 0, 0, 10, 10) == 10 * (tp["items_write_per_visible"] + tp["big_per_visible"] + tp["fill_read_per_gaussian"])
    assert bench.measured_traffic_backward("tile", 0, 0, 0, 10) == 10 * t["tile"]["scatter_write_per_gaussian"]
    assert bench.measured_traffic_backward("tile", 7, 9, 0, 0) == 7 * t["tile"]["pairs_per_hit"]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = bench.shard_views(16, rank, world)
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    h = torch.tensor([float(len(mine))], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(h, op=dist.ReduceOp.SUM)
    if rank == 0:
        out.put((t.item(), h.item()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    tmax, hsum = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert tmax == 11.0 and hsum == 16.0
