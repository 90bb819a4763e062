"""The N > 1 path of the bench (replicas, no data-path collective) on two gloo ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def test_shard_batch_partitions_the_batch():
    for batch in (1, 7, 32, 33):
        for world in (1, 2, 3, 8):
            parts = [bench.shard_batch(batch, r, world) for r in range(world)]
            flat = [s for p in parts for s in p]
            assert flat == list(range(batch))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank "times" its own replica; the job's time is the slowest rank's
    mine = 10.0 + 5.0 * rank
    worst = bench.max_over_ranks(mine, world)
    # the aggregate is steps of all ranks over that time
    out[rank] = (worst, world * 100 / (worst / 1000.0))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == (15.0, 2 * 100 / 0.015)
