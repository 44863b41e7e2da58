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


# ------------------------------------------------------------- launcher-less start and the data-parallel plan

def _rehearse(n, extra=()):
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", str(n), "--rehearse-host",
                          "--parallelism", "dp", *extra], capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    return json.loads(lines[0])


def test_bench_starts_its_own_ranks_and_plans_the_split():
    """`python bench.py --gpus 2` with no launcher starts two ranks that find each other (gloo here),
    split one cfg4 mini-batch by token count, and agree on counts, timings and merged statistics."""
    plan = _rehearse(2, ("--dw-slabs", "8"))
    assert plan["n_ranks"] == 2 and plan["parallelism"] == "dp"
    lengths = inputs.workload_lengths("cfg4_8b_bf16")
    assert sum(plan["tokens_per_rank"]) == int(lengths.sum()) == plan["global_tokens"] == int(plan["tokens_all"])
    assert sum(plan["responses_per_rank"]) == len(lengths) == plan["global_responses"]
    assert max(plan["tokens_per_rank"]) - min(plan["tokens_per_rank"]) <= int(lengths.max())
    assert plan["max_times"] == [101.0, 50.0]                # MAX over ranks of (100 + rank, 50 - rank)
    mu, sigma = plan["merged_mu_sigma"]
    assert abs(mu - 0.5) < 1e-12 and abs(sigma - 1.5) < 1e-12    # two records (mean r, M2 = 2 B_r, B_r = 64) merged
    rows = plan["dw_slab_rows"]
    assert rows[0] == 0 and rows[-1] == 151936 and len(rows) == 9 and rows == sorted(set(rows))
    assert [s[0] for s in plan["dw_slab_order"]] == list(range(8))
    assert all(lo == rows[k] and hi == rows[k + 1] for k, lo, hi in plan["dw_slab_order"])


def test_token_balanced_partition_properties():
    from paper_2509_13232_b200 import dp
    rng = np.random.default_rng(3)
    for world in (1, 2, 3, 8):
        lengths = rng.integers(1, 9000, 128)
        parts = dp.partition_by_tokens(lengths, world)
        flat = sorted(i for p in parts for i in p)
        assert flat == list(range(128)) and all(p == sorted(p) for p in parts)
        loads = [int(lengths[p].sum()) for p in parts]
        assert max(loads) - min(loads) <= int(lengths.max())
        assert dp.partition_by_tokens(lengths, world) == parts          # deterministic: every rank gets the same answer
    assert dp.partition_by_tokens([5, 5], 4) == [[0], [1], [], []]


def test_dw_slab_bounds_cover_the_vocabulary_in_whole_rounds():
    """Bookkeeping of the slab-cut dW launch (host only): the slabs tile [0, V) in order, none is empty,
    all but the last hold a whole number of rounds of CTA-pair work units."""
    from paper_2509_13232_b200 import binding as B
    from paper_2509_13232_b200 import dp
    for V, d in ((151936, 4096), (151936, 1024), (32000, 2048), (1000, 64), (256, 64)):
        for n in (1, 2, 8, 64):
            rows = B.spo_dw_slab_rows(V, d, n)
            assert rows[0] == 0 and rows[-1] == V and 1 <= len(rows) - 1 <= n
            assert all(b > a for a, b in zip(rows, rows[1:]))
            units_per_tile = -(-d // 512)
            for a, b in zip(rows[:-2], rows[1:-1]):
                assert a % 256 == 0 and b % 256 == 0
                assert ((b - a) // 256 * units_per_tile) % 74 == 0        # 74 pairs on a 148-SM device (the host default)
            assert [(k, lo, hi) for k, (lo, hi) in enumerate(zip(rows, rows[1:]))] == dp.slab_schedule(rows)
    assert B.lib().spo_dw_slab_rows(1000, 64, 0, None) == B.ERR_INVALID_ARG
    assert B.lib().spo_dw_slab_rows(1000, 64, 65, None) == B.ERR_INVALID_ARG
