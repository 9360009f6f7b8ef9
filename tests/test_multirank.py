"""The N > 1 plumbing on CPU: two gloo ranks partition the work, draw different data, and agree on
the max-reduced timing."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_08143_b200 import inputs, sharding


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import compactor_oracle as orc
        w = sharding.rank_workload(inputs.Workload("mr", 3, 2, 128, [300], [0.5], seed=5), rank)
        kp, kr, v = inputs.make_unit(w, 0, 0, 0)
        phi = inputs.make_sketch_matrix(128, 48, 0).numpy()
        s = orc.approx_leverage_scores(orc.bf16_bits_to_f64(kp.view(torch.int16).numpy()), phi)
        checksum = float(s[:10].sum())
        layers = sharding.shard_layers(5, rank, world)
        slow = sharding.max_over_ranks(10.0 + rank, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, (checksum, layers, slow))
        if rank == 0:
            out.put(gathered)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_partition_and_reduce():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (c0, l0, s0), (c1, l1, s1) = got
    assert c0 != c1                                   # ranks drew different data
    assert sorted(l0 + l1) == list(range(5)) and not set(l0) & set(l1)
    assert s0 == s1 == 11.0                           # everyone sees the slowest rank's time
    assert sharding.job_tokens_per_second(1000, 2, 10.0) == 200000.0


def test_shard_range_is_a_partition():
    for count in (0, 1, 7, 64, 513):
        for world in (1, 2, 3, 8):
            cover = []
            for r in range(world):
                b, e = sharding.shard_range(count, r, world)
                assert 0 <= b <= e <= count and e - b in (count // world, count // world + 1)
                cover += list(range(b, e))
            assert cover == list(range(count))
