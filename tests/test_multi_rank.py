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
        # each rank renders only its own streams, from the global stream index (as bench.py does with first=):
        # the pixels of a stream depend on that index alone, not on who renders it
        w = configs.batched_stress(96, 64, 128)
        frames = w.streams(S, 2, first=mine[0]).frame(1)
        local_time = 1.0 + rank                      # rank 1 is slower
        t = sharding.max_over_ranks(local_time)
        out[rank] = dict(mine=mine, gathered=gathered, t=t, rate=sharding.aggregate_rate(S * 10, world, t),
                         frames=frames.tobytes(), shape=frames.shape)
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
    # one process renders all six streams: rank r's frames are streams r * S ... r * S + S - 1 of that batch
    whole = configs.batched_stress(96, 64, 128).streams(6, 2).frame(1)
    assert whole.shape == (6, 64, 96, 3)
    for r in range(world):
        assert tuple(res[r]["shape"]) == (3, 64, 96, 3)
        assert res[r]["frames"] == whole[3 * r:3 * r + 3].tobytes()
    assert res[0]["frames"] != res[1]["frames"]                      # different streams, different pixels


def test_single_process_is_identity():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.shard_streams(0, 1, 4) == [0, 1, 2, 3]
