"""World-size-2 gloo test of the multi-rank host logic: stream sharding and max-over-ranks timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1712_01670_b200 import sharding
from paper_1712_01670_b200.synth import configs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        S = 3
        mine = sharding.shard_streams(rank, world, S)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        # each rank renders only its own streams, from the global stream index: same pixels whoever renders them
        w = configs.WORKLOADS[2]()
        frames = w.make_streams(1, 2).frame(1)
        local_time = 1.0 + rank                      # rank 1 is slower
        t = sharding.max_over_ranks(local_time)
        out[rank] = dict(mine=mine, gathered=gathered, t=t, rate=sharding.aggregate_rate(S * 10, world, t),
                         checksum=int(frames.sum()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_streams_and_reduce_time():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["mine"] == [0, 1, 2] and res[1]["mine"] == [3, 4, 5]
    flat = sorted(i for part in res[0]["gathered"] for i in part)
    assert flat == list(range(6))                                    # disjoint and complete
    assert res[0]["t"] == res[1]["t"] == 2.0                         # the slowest rank sets the time
    assert res[0]["rate"] == 3 * 10 * 2 / 2.0
    assert res[0]["checksum"] == res[1]["checksum"]                  # seeded inputs do not depend on the rank


def test_single_process_is_identity():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.shard_streams(0, 1, 4) == [0, 1, 2, 3]
