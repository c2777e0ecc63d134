"""World-size-2 run of the multi-GPU host logic on CPU (gloo): batch shards partition the images,
each rank's shard of Eq. 1 equals the corresponding slice of the whole result (b is a free index),
and timings aggregate as the max over ranks.  The per-rank compute here is the CPU oracle -- the
test is about the sharding arithmetic, not about the kernels."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1802_06905_b200 import sharding, synth


def test_shard_batch_partitions_every_batch_size():
    for B in (1, 31, 32, 64, 96, 100, 128, 250, 4096):
        for world in (1, 2, 3, 4, 8):
            covered = []
            for r in range(world):
                b0, n = sharding.shard_batch(B, world, r)
                assert n >= 0
                covered += list(range(b0, b0 + n))
                if r < world - 1:
                    assert n % 32 == 0
            assert covered == list(range(B))


def test_bench_ranks_cut_one_batch_of_world_times_b_images():
    """What `bench.py --gpus N` gives rank r: images [b0, b0+n) of ONE problem with N*B images (same
    seeded data on every rank), the Filter whole.  The shards partition the batch, their dims carry
    the shard's B, and their Image is the matching slice of the global Image."""
    import bench
    cfg = synth.CONFIGS[1]
    for world in (1, 2, 4):
        from dataclasses import replace
        glob = replace(cfg, B=cfg.B * world)
        gi, gf = synth.make_inputs(glob)
        covered = []
        for r in range(world):
            local, ib, fb, (b0, n), gB = bench.make_rank_problem(cfg, world, r)
            assert gB == cfg.B * world and local.B == n and local.dims()[1:] == cfg.dims()[1:]
            assert ib.shape == local.image_shape and fb.shape == cfg.filter_shape
            assert np.array_equal(ib, gi[..., b0:b0 + n]) and np.array_equal(fb, gf)
            covered += list(range(b0, b0 + n))
        assert covered == list(range(cfg.B * world))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, q):
    from oracle import cnn as ocnn
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cs = synth.ConvShape("shard", 96, 8, 6, 5, 4, 3, 2, 2, 1, seed=5)
    ib, fb = synth.make_inputs(cs)                     # same seeded inputs on every rank
    b0, n = sharding.shard_batch(cs.B, world, rank)
    shp = ocnn.Shape(n, cs.C, cs.K, cs.W, cs.H, cs.R, cs.S, cs.sw, cs.sh)
    out, _ = ocnn.cnn_bf16(sharding.slice_batch(ib, b0, n), fb, shp)
    # the forward needs no collective; gather only to check
    gathered = [None] * world
    dist.all_gather_object(gathered, (b0, n, out))
    t_max = sharding.max_over_ranks(1.0 + rank, dist)
    dist.barrier()
    if rank == 0:
        full, _ = ocnn.cnn_bf16(ib, fb, ocnn.Shape(*cs.dims()))
        ok = all(np.array_equal(full[..., g0:g0 + gn], gout) for g0, gn, gout in gathered)
        q.put((ok, t_max, sharding.whole_job_throughput(10.0, t_max, world)))
    dist.destroy_process_group()


def test_two_ranks_shard_the_batch_without_a_collective():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    ok, t_max, thr = q.get()
    assert ok
    assert t_max == 2.0                    # the slowest rank's time
    assert thr == pytest.approx(2 * 10.0 / 2.0)
