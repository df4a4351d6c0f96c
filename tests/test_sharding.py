"""Multi-GPU path: tokens are independent through all layers, so ranks take disjoint token ranges
and exchange nothing on the data path.  Covered here with two gloo ranks on CPU: the shards tile
the token range, and the benchmark's max-over-ranks timing reduction works."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2501_19392_b200 import synth


def test_shards_tile_the_range():
    for n in (0, 1, 127, 128, 32768, 131072, 1000003):
        for world in (1, 2, 3, 8):
            for mult in (1, 128):
                ranges = [synth.shard_range(n, r, world, mult) for r in range(world)]
                assert ranges[0][0] == 0 and ranges[-1][1] == n
                for (a, b), (c, d) in zip(ranges, ranges[1:]):
                    assert b == c and a <= b
                for a, b in ranges[:-1]:
                    assert (b - a) % mult == 0


def _worker(rank, world, port, n):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lo, hi = synth.shard_range(n, rank, world, 128)
    count = torch.tensor([hi - lo], dtype=torch.int64)
    dist.all_reduce(count, op=dist.ReduceOp.SUM)
    assert int(count) == n
    t = torch.tensor([1.0 + rank], dtype=torch.float64)       # per-rank elapsed time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert float(t) == float(world)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_partition_and_reduce():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, 32768 + 77), nprocs=2, join=True)
