"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, sharding without overlap, max-over-
ranks timing, whole-job throughput, and per-rank seeds that give different inputs."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2607_17979_b200 import dist as D, inputs as I


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, size, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(size), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    D.init("gloo")
    D.barrier()
    mine = D.shard(130, size, rank)
    times = D.max_over_ranks([10.0 + rank, 5.0 - rank])           # rank 1 slower on [0], faster on [1]
    d = I.make_config(0, trial=rank)                               # each rank draws its own sequences
    out[rank] = dict(shard=(mine.start, mine.stop), times=times, q0=int(d["q"].ravel()[0]),
                     rate=D.whole_job_rate(64.0, times[0], size))
    D.barrier()
    D.finish()


def test_two_gloo_ranks_shard_and_reduce():
    size, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(size, port, out), nprocs=size, join=True)
        r0, r1 = out[0], out[1]
    assert r0["shard"] == (0, 65) and r1["shard"] == (65, 130)      # disjoint, cover everything
    assert r0["times"] == r1["times"] == [11.0, 5.0]                # max over ranks, on both ranks
    assert r0["q0"] != r1["q0"]                                     # different seeds per rank
    assert abs(r0["rate"] - 2 * 64.0 / 11e-3) < 1e-6


def test_shard_properties():
    for n in (0, 1, 7, 64, 130):
        for size in (1, 2, 3, 8):
            parts = [D.shard(n, size, r) for r in range(size)]
            assert [i for p in parts for i in p] == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def test_single_process_helpers_need_no_process_group():
    assert D.world()[1] >= 1
    assert D.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    D.barrier()
