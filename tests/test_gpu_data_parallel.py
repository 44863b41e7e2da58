"""Data-parallel decomposition on one GPU: the mini-batch is split over two emulated ranks that run
one after the other; with the merged advantage statistics and the global denominators their losses
and dW add up to, and their dH rows equal, what the oracle gives for the whole mini-batch."""

import numpy as np
import pytest

from oracle import spo_oracle as O
from paper_2509_13232_b200 import dp, inputs
from tests.helpers import dev, oracle_loss, rel_fro, run_loss, status_word, worst_row_tile_error, ws_bytes

pytestmark = pytest.mark.gpu


def _clip_batch_dp(cfg, lengths, d, v, bf16):
    rng = np.random.default_rng(cfg)
    a = rng.standard_normal(len(lengths)).astype(np.float32)
    return inputs.loss_batch(cfg, lengths, d, v, 0.05, bf16, 0.3, target="softmax", mask_p=0.1, a_norm=a)


def _slice_batch(lb, s0, s1):
    t0, t1 = int(lb.cu_seqlens[s0]), int(lb.cu_seqlens[s1])
    return inputs.LossBatch(h=lb.h[t0:t1], w=lb.w, y=lb.y[t0:t1], logp_old=lb.logp_old[t0:t1], mask=lb.mask[t0:t1],
                            cu_seqlens=(lb.cu_seqlens[s0:s1 + 1] - lb.cu_seqlens[s0]).astype(np.int32),
                            a_norm=lb.a_norm[s0:s1], bf16=lb.bf16)


@pytest.mark.parametrize("one_pass", [False, True])
@pytest.mark.parametrize("agg", [0, 1])
def test_two_emulated_ranks_equal_the_whole_mini_batch(agg, one_pass):
    import torch
    from paper_2509_13232_b200 import binding as B
    rng = np.random.default_rng(77)
    lengths = [300, 40, 0, 520, 75, 260, 9, 410]
    n = 5000
    ab = rng.uniform(0.1, 12.0, (n, 2)).astype(np.float32)
    ids = rng.permutation(n)[:len(lengths)].astype(np.int32)
    rewards = (rng.random(len(lengths)) < 0.5).astype(np.float32)
    lb = inputs.loss_batch(78, lengths, 128, 900, 0.05, True, 0.3, target="softmax", mask_p=0.1,
                           a_norm=np.zeros(len(lengths), np.float32))
    lb.mask[int(lb.cu_seqlens[4]):int(lb.cu_seqlens[5])] = 0          # one response fully masked
    # oracle on the whole mini-batch
    raw = O.raw_advantage(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64), ids, rewards)
    a_norm, mu, sigma = O.normalise_advantages(raw, 0, 1e-8)
    lb.a_norm = a_norm.astype(np.float32)
    want = O.loss_forward(lb.h, lb.w, lb.y, lb.logp_old, lb.mask, lb.cu_seqlens, lb.a_norm, agg_mode=agg)
    want_dh, want_dw = O.loss_backward(lb.h, lb.w, lb.y, want["lse"], want["coef"])
    # two ranks: responses [0,3) and [3,8)
    splits = [(0, 3), (3, 8)]
    ab_t = dev(ab)
    p0 = B.default_params()
    recs, raws = [], []
    for s0, s1 in splits:
        a_raw = torch.empty(s1 - s0, dtype=torch.float32, device="cuda")
        a_tmp = torch.empty_like(a_raw)
        stats = torch.zeros(8, dtype=torch.float32, device="cuda")
        B.spo_advantages(ab_t, dev(ids[s0:s1]), dev(rewards[s0:s1]), a_raw, a_tmp, stats, ws_bytes(B.WS_ADVANTAGES, B=s1 - s0),
                         p0, status_word())
        torch.cuda.synchronize()
        r = stats.cpu().numpy()
        recs.append((r[0], r[3], r[2]))
        raws.append(a_raw)
    g_mu, g_m2, g_n = dp.merge_moments(recs)
    g_sigma = dp.sigma_from(g_m2, g_n, 0)
    assert abs(g_mu - mu) < 1e-6 and abs(g_sigma - sigma) < 1e-6
    seq_tok = [int(lb.mask[int(a):int(b)].sum()) for a, b in zip(lb.cu_seqlens[:-1], lb.cu_seqlens[1:])]
    n_tok, n_resp = sum(seq_tok), sum(1 for c in seq_tok if c > 0)
    params = B.default_params(agg_mode=agg, global_tokens=n_tok, global_responses=n_resp)
    loss_sum, dws, dhs = 0.0, [], []
    for (s0, s1), a_raw in zip(splits, raws):
        a_n = torch.empty_like(a_raw)
        B.spo_advantages_apply(a_raw, g_mu, g_sigma, a_n, params)
        torch.cuda.synchronize()
        np.testing.assert_allclose(a_n.cpu().numpy(), a_norm[s0:s1], rtol=1e-5, atol=2e-6)
        part = _slice_batch(lb, s0, s1)
        part.a_norm = a_n.cpu().numpy()
        got = run_loss(part, params=params, one_pass=one_pass)
        assert got["status"] == 0
        loss_sum += got["loss"]
        dws.append(got["dW"])
        dhs.append(got["dH"])
    assert abs(loss_sum - want["loss"]) <= 2e-3
    assert rel_fro(np.concatenate(dhs, 0), want_dh) <= 1e-2
    assert rel_fro(dws[0] + dws[1], want_dw) <= 1e-2


def _fwd_bwd(lb, params, events=None):
    """One spo_loss_fwd_bwd (or, with events, spo_loss_fwd_bwd_slabs) call; returns (loss, dH, dW) tensors."""
    import torch
    from paper_2509_13232_b200 import binding as B
    H, W = dev(lb.h, torch.bfloat16), dev(lb.w, torch.bfloat16)
    T, d = H.shape
    V, S = W.shape[0], len(lb.cu_seqlens) - 1
    f32 = dict(dtype=torch.float32, device="cuda")
    loss = torch.zeros(4, **f32)
    logp, lse, coef = (torch.zeros(T, **f32) for _ in range(3))
    dH = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
    dW = torch.full((V, d), float("nan"), **f32)
    st = status_word()
    args = (H, W, dev(lb.y), dev(lb.logp_old), dev(lb.mask), dev(lb.cu_seqlens), dev(lb.a_norm), 1.0, loss, logp, lse,
            coef, None, dH, dW, 0, ws_bytes(B.WS_LOSS_FWD_BWD, T=T, d=d, V=V, B=S), params, st)
    if events is None:
        B.spo_loss_fwd_bwd(*args)
    else:
        B.spo_loss_fwd_bwd_slabs(*args, events)
    return loss, dH, dW, st


@pytest.mark.parametrize("lengths", [[700, 40, 520, 75], [5000, 4400, 9000, 1600]])
def test_slab_cut_last_dw_contraction_is_bitwise_the_plain_call_and_reduces_in_slab_order(lengths):
    """The data-parallel variant cuts the last dW launch into vocabulary slabs with an event behind
    each.  One chunk and three chunks (the slabs belong to the last group of chunks only): results
    equal spo_loss_fwd_bwd bit for bit, and two emulated ranks whose dW are added slab by slab, each
    slab as soon as its event has passed on a second stream, give the whole mini-batch's dW."""
    import torch
    from paper_2509_13232_b200 import binding as B
    v, d = 20000, 1024                      # 79 vocabulary row tiles, two hidden column tiles: slabs of 37 row tiles
    small = sum(lengths) < 5000
    if small:
        lb = inputs.loss_batch(79, lengths, d, v, 0.02, True, 0.3, target="softmax", mask_p=0.1)
    else:                                   # three chunks: too many logits for the host, generated on the device
        data = inputs.loss_batch_device(79, np.asarray(lengths), d, v, 0.02, 0.3, torch.device("cuda", 0))
        rng = inputs.rng_for(79, 5)
        lb = inputs.LossBatch(h=data["h"].float().cpu().numpy(), w=data["w"].float().cpu().numpy(),
                              y=data["y"].cpu().numpy(), logp_old=data["logp_old"].cpu().numpy(),
                              mask=(rng.random(data["T"]) >= 0.1).astype(np.uint8),
                              cu_seqlens=data["cu_seqlens"].cpu().numpy(),
                              a_norm=rng.standard_normal(len(lengths)).astype(np.float32), bf16=True)
    params = B.default_params()
    plain = _fwd_bwd(lb, params)
    rows = B.spo_dw_slab_rows(v, d, 6)
    assert len(rows) - 1 == 3
    red = dp.SlabAllReduce(rows, torch.device("cuda", 0))
    cut = _fwd_bwd(lb, params, red.events)
    red.reduce(cut[2])                       # one process: waits for every slab's event, no collective
    red.finish()
    torch.cuda.synchronize()
    assert int(plain[3][0].item()) == 0 and int(cut[3][0].item()) == 0
    for a, b in zip(plain[:3], cut[:3]):
        assert torch.equal(a, b)
    # two ranks, one after the other, each with the whole batch's denominators
    n_tok, s_mid = int(lb.mask.sum()), 2
    pg = B.default_params(global_tokens=n_tok, global_responses=len(lengths))
    total = torch.zeros_like(plain[2])
    side = torch.cuda.Stream()
    for s0, s1 in ((0, s_mid), (s_mid, len(lengths))):
        part = _slice_batch(lb, s0, s1)
        evs = dp.SlabAllReduce(rows, torch.device("cuda", 0))
        loss, dH, dW, st = _fwd_bwd(part, pg, evs.events)
        with torch.cuda.stream(side):
            for k, lo, hi in dp.slab_schedule(rows):
                side.wait_event(evs.events[k])        # rows lo..hi of this rank's dW are final from here on
                total[lo:hi] += dW[lo:hi]
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        assert int(st[0].item()) == 0
    assert rel_fro(total.cpu().numpy(), plain[2].cpu().numpy()) <= 2e-3
    if small:                               # ... and the oracle's, where the host can form the logits
        want = O.loss_forward(lb.h, lb.w, lb.y, lb.logp_old, lb.mask, lb.cu_seqlens, lb.a_norm)
        _, want_dw = O.loss_backward(lb.h, lb.w, lb.y, want["lse"], want["coef"])
        assert rel_fro(total.cpu().numpy(), want_dw) <= 1e-2


def test_data_parallel_step_with_one_rank_equals_the_plain_step():
    """The step bench.py runs under `--parallelism dp` (rewards put together over the ranks, whole-batch
    advantages and tracker update on every rank, global denominators, slab-cut loss call with the
    reductions behind the events) on a process group of ONE rank: every exchange is the identity, so
    every output must equal the plain step's bit for bit.  (More ranks cannot run here; their host
    logic is covered on gloo ranks.)"""
    import os
    import socket
    import torch
    import torch.distributed as dist
    import bench
    dev0 = torch.device("cuda", 0)
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev0)
    try:
        plain = bench.Step("cfg3_small_bf16", dev0, 0)
        plain.run()
        torch.cuda.synchronize()
        keep = [t.clone() for t in (plain.loss, plain.logp, plain.coef, plain.dH, plain.dW, plain.ids, plain.ab,
                                    plain.a_norm)]
        assert int(plain.status[0].item()) == 0
        del plain
        torch.cuda.empty_cache()
        part = bench.Step("cfg3_small_bf16", dev0, 0, dp_world=1, dw_slabs=8)
        assert len(part.reducer.events) >= 2 and part.my_responses.tolist() == list(range(part.S_all))
        part.run()
        torch.cuda.synchronize()
        assert int(part.status[0].item()) == 0
        for a, b in zip(keep, (part.loss, part.logp, part.coef, part.dH, part.dW, part.ids, part.ab, part.a_norm)):
            assert torch.equal(a, b)
        del part
        torch.cuda.empty_cache()
        # the same step with dW scattered into per-rank shards (one shard here): the sums are formed by
        # store-reductions on top of a zeroed shard, so dW agrees to rounding instead of bit for bit
        scat = bench.Step("cfg3_small_bf16", dev0, 0, dp_world=1, dw_reduce="scatter")
        scat.run()
        torch.cuda.synchronize()
        assert int(scat.status[0].item()) == 0
        for a, b in zip(keep[:4] + keep[5:], (scat.loss, scat.logp, scat.coef, scat.dH, scat.ids, scat.ab, scat.a_norm)):
            assert torch.equal(a, b)
        assert scat.shards.local.shape == keep[4].shape
        assert rel_fro(scat.shards.local.cpu().numpy(), keep[4].cpu().numpy()) <= 1e-6
    finally:
        dist.destroy_process_group()


def _scatter_call(lb, params, shards, dw_init=None):
    """One spo_loss_fwd_bwd_scatter call; returns (loss, dH, dW scratch, status)."""
    import torch
    from paper_2509_13232_b200 import binding as B
    tdt = torch.bfloat16 if lb.bf16 else torch.float32
    H, W = dev(lb.h, tdt), dev(lb.w, tdt)
    T, d = H.shape
    V, S = W.shape[0], len(lb.cu_seqlens) - 1
    f32 = dict(dtype=torch.float32, device="cuda")
    loss = torch.zeros(4, **f32)
    logp, lse, coef = (torch.zeros(max(T, 1), **f32) for _ in range(3))
    dH = torch.zeros((max(T, 1), d), dtype=tdt, device="cuda")
    dW = torch.full((V, d), float("nan"), **f32) if dw_init is None else dev(dw_init).clone()
    st = status_word()
    B.spo_loss_fwd_bwd_scatter(H, W, dev(lb.y), dev(lb.logp_old), dev(lb.mask), dev(lb.cu_seqlens), dev(lb.a_norm), 1.0,
                               loss, logp, lse, coef, None, dH[:T], dW, 0 if dw_init is None else 1,
                               ws_bytes(B.WS_LOSS_FWD_BWD, T=T, d=d, V=V, B=S), params, st, shards)
    return loss, dH, dW, st


@pytest.mark.parametrize("case", ["one_chunk", "three_chunks", "fp32", "gspo"])
def test_reduce_scatter_form_two_emulated_ranks_fill_the_owners_shards(case):
    """spo_loss_fwd_bwd_scatter: two ranks, one after the other on this GPU, each with its part of the
    mini-batch and the whole batch's denominators, add their dW into three shards (local buffers standing
    in for the owners' memory; the last shard is ragged).  Together the shards must hold the dW that one
    plain call on the whole mini-batch gives; loss and dH are untouched by the variant."""
    import torch
    from paper_2509_13232_b200 import binding as B
    bf16 = case != "fp32"
    if case == "three_chunks":
        lengths, d, v = [5000, 4400, 9000, 1600], 128, 3000
    elif case == "fp32":
        lengths, d, v = [30, 4, 51, 9], 32, 257
    else:
        lengths, d, v = [700, 40, 520, 75], 128, 3000
    lb = _clip_batch_dp(160, lengths, d, v, bf16)
    sur = B.SUR_GSPO if case == "gspo" else B.SUR_PPO_CLIP
    n_tok = int(lb.mask.sum())
    n_resp = sum(1 for a, b in zip(lb.cu_seqlens[:-1], lb.cu_seqlens[1:]) if lb.mask[int(a):int(b)].any())
    whole = run_loss(lb, params=B.default_params(surrogate=sur), one_pass=True)
    rows_per = -(-v // 3) + 5                                   # 3 shards, the last one shorter
    bufs = [torch.zeros((rows_per, d), dtype=torch.float32, device="cuda") for _ in range(3)]
    shards = B.dw_shards(bufs, rows_per)
    pg = B.default_params(surrogate=sur, global_tokens=n_tok, global_responses=n_resp)
    loss_sum, dhs = 0.0, []
    for s0, s1 in ((0, 2), (2, len(lengths))):
        part = _slice_batch(lb, s0, s1)
        loss, dH, _, st = _scatter_call(part, pg, shards)
        torch.cuda.synchronize()
        assert int(st[0].item()) == 0
        loss_sum += float(loss[0].item())
        dhs.append(dH[:part.h.shape[0]].float().cpu().numpy())
    got_dw = torch.cat(bufs, 0)[:v].cpu().numpy()
    assert float(torch.cat(bufs, 0)[v:].abs().max().item()) == 0.0      # rows past the vocabulary stay untouched
    tol = 2e-3 if bf16 else 1e-5
    assert rel_fro(got_dw, whole["dW"]) <= tol
    assert abs(loss_sum - whole["loss"]) <= (2e-3 if bf16 else 1e-5)
    assert rel_fro(np.concatenate(dhs, 0), whole["dH"]) <= tol
    want = oracle_loss(lb, params=B.default_params(surrogate=sur))     # and the float64 definition of the whole batch
    assert rel_fro(got_dw, want["dW"]) <= (1e-2 if bf16 else 1e-4)
    assert worst_row_tile_error(got_dw, want["dW"])[0] <= (2e-2 if bf16 else 1e-4)
    assert abs(loss_sum - want["loss"]) <= (2e-3 if bf16 else 1e-5)


def test_peer_shards_on_a_one_rank_group_hold_the_plain_dw():
    """dp.PeerShards (shards in memory mapped into every rank of the group) with a group of one rank: the
    table has one shard, this rank's, and after begin_step / the scatter call / end_step it holds the dW
    of the plain call.  (Shards in a peer's memory need a second GPU.)"""
    import os
    import socket
    import torch
    import torch.distributed as dist
    from paper_2509_13232_b200 import binding as B
    dev0 = torch.device("cuda", 0)
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev0)
    try:
        d, v = 128, 3000
        lb = _clip_batch_dp(161, [700, 40, 520, 75], d, v, True)
        whole = run_loss(lb, params=B.default_params(), one_pass=True)
        shards = dp.PeerShards(v, d, dev0)
        assert shards.rows_per_shard == v and shards.table.n_shards == 1
        for _ in range(2):                                     # a second step starts from a zeroed shard again
            shards.begin_step()
            _, _, _, st = _scatter_call(lb, B.default_params(), shards.table)
            shards.end_step()
            torch.cuda.synchronize()
            assert int(st[0].item()) == 0
            assert rel_fro(shards.local.cpu().numpy(), whole["dW"]) <= 2e-3
    finally:
        dist.destroy_process_group()
