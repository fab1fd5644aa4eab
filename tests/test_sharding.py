"""N>1 bookkeeping on CPU: two gloo ranks shard utterances, draw rank-specific inputs and
reduce the step time by max over ranks (the only communication of the path)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2206_07882_b200 import sharding, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lo, hi = sharding.shard_range(13, rank, world)
    mel = synth.logmel(sharding.rank_seed(4, rank), 2, 8, 4)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    rtf = sharding.aggregate_rtf(local_ms, utterances_per_rank=64, seconds_per_utterance=10.0, world=world)
    out[rank] = (lo, hi, float(mel.sum()), rtf, sharding.job_time_ms(local_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_and_reduce():
    world = 2
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    (lo0, hi0, s0, rtf0, t0), (lo1, hi1, s1, rtf1, t1) = out[0], out[1]
    assert (lo0, hi0, lo1, hi1) == (0, 7, 7, 13)           # disjoint, covering, balanced
    assert s0 != s1                                         # every rank has its own utterances
    assert t0 == t1 == 15.0                                 # max over ranks
    assert rtf0 == rtf1 == (15.0 / 1e3) / (2 * 64 * 10.0)   # whole-job audio in the denominator


def test_shard_range_properties():
    for n in (0, 1, 7, 64, 1000):
        for world in (1, 2, 3, 8):
            parts = [sharding.shard_range(n, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == n
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.job_time_ms(3.5) == 3.5                 # no process group: identity
