"""World-size-2 check (gloo, CPU) of the only exchange the data-parallel path has: every rank must end up
with the element-wise MAX of the calibration maxima, and the batch shards must tile the batch exactly."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1805_08691_b200 import pipeline
    local = {"x": 1.0 + rank, "a": 5.0 - rank, "b": 0.25, "c": 3.0 * (rank + 1)}
    merged = pipeline.sync_maxima(local)
    out[rank] = (merged, pipeline.shard_batch(33, rank, world))
    dist.destroy_process_group()


def test_maxima_are_reduced_with_max_and_shards_tile_the_batch():
    world = 2
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    want = {"x": 2.0, "a": 5.0, "b": 0.25, "c": 6.0}
    assert out[0][0] == want and out[1][0] == want
    (b0, e0), (b1, e1) = out[0][1], out[1][1]
    assert b0 == 0 and e0 == b1 and e1 == 33 and abs((e0 - b0) - (e1 - b1)) <= 1


def test_sync_is_identity_without_a_process_group():
    from paper_1805_08691_b200 import pipeline
    m = {"x": 1.5, "y": 0.0}
    assert pipeline.sync_maxima(m) == m
    assert pipeline.shard_batch(8, 0, 1) == (0, 8)
