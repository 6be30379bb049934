"""The N > 1 path is replicas only: sequence sharding and the max-over-ranks / sum-over-ranks reduction,
exercised with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2302_01318_b200 import replicas


def test_shards_partition_the_sequences():
    for n in (0, 1, 7, 16):
        for w in (1, 2, 3, 8):
            got = sorted(i for r in range(w) for i in replicas.shard_sequences(n, r, w))
            assert got == list(range(n))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = replicas.shard_sequences(5, rank, world)
    secs, toks = replicas.job_time_and_tokens(1.0 + rank, 128 * len(mine), dist)
    out[rank] = (secs, toks, mine)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_time_and_tokens():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0][:2] == out[1][:2] == (2.0, 128 * 5)
    assert out[0][2] == [0, 2, 4] and out[1][2] == [1, 3]
