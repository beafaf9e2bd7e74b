"""Batch-sharded replicas on two CPU ranks (gloo): clip sharding, max-over-ranks timing and
whole-job throughput aggregation used by the benchmark when it runs on several GPUs."""
import os
import socket

import torch.multiprocessing as mp

from paper_2007_09835_b200 import dist


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    g = dist.init(world, rank, "gloo")
    clips = dist.shard_clips(9, world, rank)
    dist.barrier(g)
    slow = dist.max_over_ranks(10.0 + 5.0 * rank, g)
    thr = dist.aggregate_throughput(float(len(clips)), 10.0 + 5.0 * rank, g)
    out[rank] = (list(clips), slow, thr)
    dist.shutdown(g)


def test_two_rank_sharding_and_aggregation():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == [0, 1, 2, 3, 4] and res[1][0] == [5, 6, 7, 8]      # disjoint, complete
    for r in range(world):
        assert res[r][1] == 15.0                                            # slowest rank decides
        assert abs(res[r][2] - 9 / 15e-3) < 1e-6                            # all clips / slowest time


def test_shard_clips_covers_everything():
    for n in (1, 7, 8, 16, 33):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in dist.shard_clips(n, world, r)]
            assert got == list(range(n))


def test_single_process_is_identity():
    assert dist.max_over_ranks(3.5, None) == 3.5
    assert dist.aggregate_throughput(8.0, 2.0, None) == 4000.0
