"""Two CPU ranks over gloo: the bookkeeping that bench.py --gpus N relies on."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import synth_inputs as S
from paper_2511_20564_b200 import replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank reports its own time and work; rank 1 is the slow one
        times, counts = replicas.reduce_measurements([0.5 + rank, 2.0 - rank], [100 * (rank + 1), 7])
        first = replicas.first_step_of(rank)
        batch = S.seed_batch(1000, 16, 3, first)
        gathered = [None] * world
        dist.all_gather_object(gathered, batch.tolist())
        out[rank] = (times, counts, gathered)
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_to_slowest_time_and_total_work():
    world = 2
    port = 29500 + (os.getpid() % 1000)
    with mp.get_context("spawn").Manager() as m:        # spawn: earlier tests may have started OpenMP threads here
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            times, counts, gathered = out[rank]
            assert times == [1.5, 2.0]                 # max over ranks, per entry
            assert counts == [300, 14]                 # sum over ranks
            assert gathered[0] != gathered[1]          # the ranks train on different batches
            assert gathered[0] == S.seed_batch(1000, 16, 3, 0).tolist()


def test_single_process_passes_through():
    assert replicas.reduce_measurements([1.25], [3]) == ([1.25], [3])
    assert replicas.first_step_of(3) == 3_000_000
