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


def _dp_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2509_13232_b200 import dp
        rng = np.random.default_rng(5)
        full = rng.uniform(-1, 1, 1000)
        mine = full[:300] if rank == 0 else full[300:]
        rec = torch.tensor([mine.mean(), mine.std(), len(mine), ((mine - mine.mean()) ** 2).sum()], dtype=torch.float32)
        mu, sigma = dp.global_advantage_stats(rec, ddof=0)
        ntok, nresp = dp.global_counts(100 * (rank + 1), 3 + rank)
        dw = torch.full((4,), float(rank + 1))
        dp.allreduce_sum(dw)
        out[rank] = (mu, sigma, ntok, nresp, dw.tolist(), float(full.mean()), float(full.std()))
    finally:
        dist.destroy_process_group()


def test_data_parallel_glue_merges_statistics_and_counts():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_dp_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    for rank in range(world):
        mu, sigma, ntok, nresp, dw, want_mu, want_sigma = out[rank]
        assert abs(mu - want_mu) < 1e-6 and abs(sigma - want_sigma) < 1e-6
        assert (ntok, nresp) == (300, 7)
        assert dw == [3.0] * 4


def test_merge_moments_is_exact_for_any_grouping():
    from paper_2509_13232_b200 import dp
    rng = np.random.default_rng(6)
    x = rng.normal(0.3, 2.0, 997)
    cuts = [0, 1, 50, 51, 400, 997]
    parts = [(x[a:b].mean(), ((x[a:b] - x[a:b].mean()) ** 2).sum(), b - a) for a, b in zip(cuts[:-1], cuts[1:])]
    parts.insert(2, (0.0, 0.0, 0))                       # an empty rank
    mean, m2, n = dp.merge_moments(parts)
    assert n == 997 and abs(mean - x.mean()) < 1e-12
    assert abs(dp.sigma_from(m2, n, 0) - x.std()) < 1e-12 and abs(dp.sigma_from(m2, n, 1) - x.std(ddof=1)) < 1e-12
