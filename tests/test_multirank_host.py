"""Host logic of the N > 1 benchmark path on CPU ranks (gloo, world size 2): ranks are
independent replicas, timings reduce with MAX, tokens with SUM, and every rank draws its own
mini-batch from its own seed."""

import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2509_13232_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        times = [10.0 + rank, 5.0 - rank, 1.0]
        tokens = 1000 * (rank + 1)
        red, tok = bench.reduce_over_ranks(times, tokens, world, torch.device("cpu"))
        tb = inputs.tracker_batch(40 + rank, 1000, 16, 32)
        out[rank] = (red, tok, tb.ids.tolist())
    finally:
        dist.destroy_process_group()


def test_max_of_times_sum_of_tokens_and_distinct_batches():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    for rank in range(world):
        red, tok, _ = out[rank]
        assert red == [11.0, 5.0, 1.0]
        assert tok == 3000.0
    assert out[0][2] != out[1][2]


def test_single_rank_is_identity():
    red, tok = bench.reduce_over_ranks([3.0, 4.0], 7, 1, torch.device("cpu"))
    assert red == [3.0, 4.0] and tok == 7.0
    assert np.isfinite(red).all()
