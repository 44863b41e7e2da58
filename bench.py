#!/usr/bin/env python
"""Benchmark of the SPO hot path on B200.

One "step" is one pass of the whole path over one synthetic mini-batch:
prioritised sampling -> advantages (pre-update baseline) + normalisation ->
tracker update -> fused loss forward + backward (loss, logp, lse, coef, dH, dW).
The loss runs as the one-pass call spo_loss_fwd_bwd (three LM-head contractions per
token) by default, or as spo_loss_fwd followed by spo_loss_bwd with `--path split`
(four: the backward recomputes the logits).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints one JSON line (rank 0).  `value` is response tokens/s with inputs resident
in HBM; `e2e` is the same step fed from pinned host buffers with the copies inside
the timed region.  `--impl reference` times the float64 CPU oracle on a bounded
sample of the same workload instead.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "response tokens/s, fused SPO loss fwd+bwd (d4096,V151936,bf16); % bf16 peak"
UNIT = "tokens/s"
TABLE_N = 1_000_000          # tracker table the step samples from and updates
# DRAM read+write bytes (dram__bytes_read.sum + dram__bytes_write.sum) of all launches of one cfg4 step:
# one chunk's launches captured with ncu on a slice of the workload, times the chunks of a step.
# None = the kernels of that path changed after the counters were taken.
CFG4_STEP_DRAM_BYTES = {"split": 9.19e11, "onepass": 6.9e11}
DW_CHUNK_GROUP = 2           # chunks of token rows whose dW contraction shares one launch (the library's constant)

LOSS_SHAPES = {
    # workload: (d, V, w_std, old-logprob noise, reward probability)
    "cfg3_small_bf16": (1024, 151936, 0.02, 0.02, 0.4),
    "cfg4_8b_bf16": (4096, 151936, 0.02, 0.02, 0.3),
    "cfg5_longtail_bf16": (4096, 151936, 0.02, 0.02, 0.3),
}
# prompts in the tracker table of each workload (cfg5 names a 100 000-prompt table)
TABLE_PROMPTS = {"cfg5_longtail_bf16": 100_000}


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"tflops": float(p["bf16_tflops_sustained"]), "tflops_burst": float(p["bf16_tflops"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    except Exception:
        return {"tflops": 1400.0, "tflops_burst": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self._stop = threading.Event()
        self._thr = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5)
                parts = [x.strip() for x in out.stdout.strip().split(",")]
                if len(parts) == 6:
                    self.rows.append(parts)
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thr.join(timeout=6)

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        sm = sorted(float(r[0]) for r in self.rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(self.rows[0][1]), "reasons": reasons,
                "samples": len(self.rows)}


class Step:
    """Device buffers of one workload and the call sequence of one step."""

    def __init__(self, workload, device, rank, responses=None, custom=None, mask_frac=0.0, path="onepass",
                 entropy=False, dp_world=None, dw_slabs=8, surrogate="ppo_clip", dual_clip=0.0, dw_reduce="allreduce"):
        """dp_world = N: this rank holds its share of ONE mini-batch split over N ranks by token count
        (W and the tracker table replicated); None: the rank has a mini-batch of its own.
        dw_reduce: "allreduce" sums dW over the ranks slab by slab behind the last contraction (every rank
        ends with the whole dW); "scatter" has that contraction add its tiles into the vocabulary shard of
        the owning rank's memory (every rank ends with its rows of dW in self.shards.local)."""
        import torch
        from paper_2509_13232_b200 import binding as B
        from paper_2509_13232_b200 import dp, inputs
        self.B, self.torch = B, torch
        self.dp_world = dp_world
        if custom:                       # T,d,V: eight equal responses, weights scaled to unit-variance logits
            t_c, d, V = custom
            w_std, noise, rew_p = 1.3 / d ** 0.5, 0.02, 0.3
            lengths = np.full(8, t_c // 8, dtype=np.int64)
            lengths[-1] += t_c - int(lengths.sum())
            cfg = 9
        else:
            d, V, w_std, noise, rew_p = LOSS_SHAPES[workload]
            lengths = inputs.workload_lengths(workload)
            if responses:
                lengths = lengths[:responses]
            cfg = int(workload[3])
        batch_cfg = cfg * 10 if dp_world else cfg * 10 + rank     # what the table, uniforms and W are seeded by
        self.S_all = len(lengths)
        self.n_tok_all = int(np.sum(lengths))
        self.my_responses = None
        if dp_world:
            self.my_responses = np.asarray(dp.partition_by_tokens(lengths, dp_world)[rank], dtype=np.int64)
            lengths = np.asarray(lengths)[self.my_responses]
        data = inputs.loss_batch_device(cfg * 10 + rank, lengths, d, V, w_std, noise, device, adv_p=rew_p,
                                        w_cfg=batch_cfg)
        self.data = data
        self.T, self.d, self.V, self.S = data["T"], d, V, data["S"]
        self.mask_frac = float(mask_frac)
        self.onepass = path == "onepass"
        if self.mask_frac > 0.0:
            # contiguous masked spans inside the responses, the way tool output sits inside a
            # tool-integrated-reasoning response: spans of 32..256 tokens until the share is reached
            rng = inputs.rng_for(cfg * 10 + rank, 7)
            m = np.ones(self.T, dtype=np.uint8)
            while 1.0 - m.mean() < self.mask_frac:
                a = int(rng.integers(0, self.T))
                m[a:a + int(rng.integers(32, 257))] = 0
            data["mask"] = torch.from_numpy(m).to(device)
        self.n_tok = int(data["mask"].sum().item())
        self.table_n = TABLE_PROMPTS.get(workload, TABLE_N)
        tb = inputs.tracker_batch(batch_cfg, self.table_n, self.S_all, 2 * self.S_all)
        f32 = dict(dtype=torch.float32, device=device)
        self.ab0 = torch.from_numpy(tb.ab).to(device)
        self.ab = self.ab0.clone()
        self.kl_table = torch.from_numpy(tb.kl_table).to(device)
        self.uniforms = torch.from_numpy(tb.uniforms).to(device)
        self.rewards = data["rewards"]
        self.params = B.default_params(surrogate={"ppo_clip": B.SUR_PPO_CLIP, "cispo": B.SUR_CISPO,
                                                  "gspo": B.SUR_GSPO}[surrogate], dual_clip=float(dual_clip))
        self.ids = torch.empty(self.S_all, dtype=torch.int32, device=device)
        self.a_norm_all = torch.empty(self.S_all, **f32)      # one value per response of the whole mini-batch
        self.a_norm = self.a_norm_all                         # ... and of this rank's responses
        if dp_world:
            # every rank owns the rewards of its own responses; the full vector is put together each step
            self.my_idx = torch.from_numpy(self.my_responses).to(device)
            self.rewards_all = torch.zeros(self.S_all, **f32)
            self.a_norm = torch.empty(self.S, **f32)
            self.params.global_tokens = self.n_tok_all        # denominators of the whole mini-batch (mask is all ones)
            self.params.global_responses = self.S_all
            self.shards = dp.PeerShards(V, d, device) if dw_reduce == "scatter" else None
            self.reducer = None if self.shards else dp.SlabAllReduce(B.spo_dw_slab_rows(V, d, dw_slabs), device)
        self.stats = torch.empty(8, **f32)
        self.loss = torch.zeros(4, **f32)
        self.logp, self.lse, self.coef = (torch.empty(self.T, **f32) for _ in range(3))
        self.entropy = torch.empty(self.T, **f32) if entropy else None      # optional per-token policy entropy
        self.dH = torch.empty((self.T, d), dtype=torch.bfloat16, device=device)
        self.dW = torch.empty((V, d), **f32)
        self.status = torch.zeros(4, dtype=torch.int32, device=device)
        u8 = dict(dtype=torch.uint8, device=device)
        self.ws_sample = torch.empty(B.spo_workspace_bytes(B.WS_SAMPLE, N=self.table_n, M=2 * self.S_all), **u8)
        self.ws_adv = torch.empty(B.spo_workspace_bytes(B.WS_ADVANTAGES, B=self.S_all), **u8)
        self.ws_bwd_bytes = B.spo_workspace_bytes(B.WS_LOSS_BWD, T=self.T, d=d, V=V)
        if self.mask_frac > 0.0:        # row lists: unmasked rows (one-pass) or rows with gradient (split backward)
            self.rows = torch.empty(self.T, dtype=torch.int32, device=device)
            self.n_active = torch.zeros(4, dtype=torch.int32, device=device)
            self.ws_rows = torch.empty(B.spo_workspace_bytes(B.WS_ACTIVE_ROWS, T=self.T), **u8)
        if self.onepass and self.mask_frac > 0.0:
            self.ws_loss = torch.empty(B.spo_workspace_bytes(B.WS_LOSS_FWD_BWD_ROWS, T=self.n_tok, d=d, V=V, B=self.S),
                                       **u8)
        elif self.onepass:
            self.ws_loss = torch.empty(B.spo_workspace_bytes(B.WS_LOSS_FWD_BWD, T=self.T, d=d, V=V, B=self.S), **u8)
        else:
            self.ws_fwd = torch.empty(B.spo_workspace_bytes(B.WS_LOSS_FWD, T=self.T, d=d, V=V, B=self.S), **u8)
            if self.mask_frac > 0.0:    # backward over the rows with gradient only
                self.ws_bwd = torch.empty(B.spo_workspace_bytes(B.WS_LOSS_BWD_ROWS, T=self.n_tok, d=d, V=V), **u8)
            else:
                self.ws_bwd = torch.empty(self.ws_bwd_bytes, **u8)
        chunk_rows = self.ws_bwd_bytes // (((V + 255) // 256) * 256 * 2)
        self.bwd_chunks = -(-self.T // chunk_rows)
        # kernels launched by one step: sampling 4 (tile sums, their prefix, search, accept; 3 for tables above
        # 2^20 prompts), advantages + update 1, then
        # split path: forward 3 (count, contraction, finalise), backward 3 per chunk;
        # one-pass path: count 1, first-tile pass 1, per chunk 4 (logits contraction, finalise, row scaling
        # of H, dH) and one dW contraction per DW_CHUNK_GROUP chunks.  Memsets are not counted.
        self.flops_fwd = 2.0 * self.T * d * V
        n_samp = 4 if self.table_n <= (1 << 20) else 3
        chunks_act = -(-self.n_tok // chunk_rows)          # chunks of the compacted batch (masked workloads)
        if self.onepass and self.mask_frac > 0.0:
            # row list 3, gather 1, boundaries 1, one-pass on the compacted batch, two scatters
            self.launches = n_samp + 1 + 3 + 1 + 1 + (2 + 4 * chunks_act + -(-chunks_act // DW_CHUNK_GROUP)) + 2
            self.flops_fwd = 2.0 * self.n_tok * d * V
            self.flops_bwd = 4.0 * self.n_tok * d * V
        elif self.onepass:
            self.launches = n_samp + 1 + 2 + 4 * self.bwd_chunks + -(-self.bwd_chunks // DW_CHUNK_GROUP)
            self.flops_bwd = 4.0 * self.T * d * V
        elif self.mask_frac > 0.0:
            # forward over all rows; row list 3, gather 1, backward on the rows with gradient, scatter 1
            self.launches = n_samp + 1 + 3 + 3 + 1 + 3 * chunks_act + 1
            self.flops_bwd = 6.0 * self.n_tok * d * V
        else:
            self.launches = n_samp + 1 + 3 + 3 * self.bwd_chunks
            self.flops_bwd = 6.0 * self.T * d * V
        if dp_world and self.reducer is not None:
            self.launches += len(self.reducer.events) - 1      # the last dW contraction runs as one launch per slab

    def small(self):
        B = self.B
        B.spo_sample_prompts(self.ab, self.uniforms, self.S_all, self.ids, None, self.ws_sample, self.params, self.status)
        rewards = self.rewards
        if self.dp_world:
            # the table is replicated and every rank applies the whole batch's updates, so the rewards of
            # all responses are needed everywhere: scatter this rank's into a zero vector and sum over ranks
            # (S floats).  With them every rank also forms the batch-global normalisation by itself.
            import torch.distributed as dist
            self.rewards_all.zero_()
            self.rewards_all.index_copy_(0, self.my_idx, self.rewards)
            dist.all_reduce(self.rewards_all)
            rewards = self.rewards_all
        # raw advantage (pre-update baseline), tracker update and normalisation in one pass over the entries
        B.spo_advantages_update(self.ab, self.ids, rewards, self.kl_table, 1, None, self.a_norm_all, self.stats,
                                self.ws_adv, self.params, self.status)
        if self.dp_world:
            self.torch.index_select(self.a_norm_all, 0, self.my_idx, out=self.a_norm)

    def fwd(self, h=None, y=None, logp_old=None, mask=None, cu=None):
        D = self.data
        self.B.spo_loss_fwd(D["h"] if h is None else h, D["w"], D["y"] if y is None else y,
                            D["logp_old"] if logp_old is None else logp_old, D["mask"] if mask is None else mask,
                            D["cu_seqlens"] if cu is None else cu, self.a_norm, self.loss, self.logp, self.lse,
                            self.coef, None, self.ws_fwd, self.params, self.status, entropy=self.entropy)

    def bwd(self, h=None, y=None):
        D = self.data
        if self.mask_frac > 0.0:
            B = self.B
            B.spo_loss_active_rows(self.coef, self.rows, self.n_active, self.ws_rows)
            n_act = int(self.n_active[0].item())          # the one host read-back of this path
            B.spo_loss_bwd_rows(D["h"] if h is None else h, D["w"], D["y"] if y is None else y, self.lse, self.coef,
                                1.0, self.rows, n_act, self.dH, self.dW, 0, self.ws_bwd, self.params, self.status)
            return
        self.B.spo_loss_bwd(D["h"] if h is None else h, D["w"], D["y"] if y is None else y, self.lse, self.coef,
                            1.0, self.dH, self.dW, 0, self.ws_bwd, self.params, self.status)

    def loss_onepass(self, h=None, y=None, logp_old=None, mask=None, cu=None):
        D = self.data
        if self.mask_frac > 0.0:        # the unmasked rows only
            B = self.B
            B.spo_loss_mask_rows(D["mask"] if mask is None else mask, self.rows, self.n_active, self.ws_rows)
            n_act = int(self.n_active[0].item())          # the one host read-back of this path
            B.spo_loss_fwd_bwd_rows(D["h"] if h is None else h, D["w"], D["y"] if y is None else y,
                                    D["logp_old"] if logp_old is None else logp_old,
                                    D["cu_seqlens"] if cu is None else cu, self.a_norm, self.rows, n_act, 1.0,
                                    self.loss, self.logp, self.lse, self.coef, None, self.dH, self.dW, 0, self.ws_loss,
                                    self.params, self.status)
            return
        args = (D["h"] if h is None else h, D["w"], D["y"] if y is None else y,
                D["logp_old"] if logp_old is None else logp_old, D["mask"] if mask is None else mask,
                D["cu_seqlens"] if cu is None else cu, self.a_norm, 1.0, self.loss, self.logp,
                self.lse, self.coef, None, self.dH, self.dW, 0, self.ws_loss, self.params, self.status)
        if self.dp_world:
            # the ranks' dW and loss add up to the mini-batch's; dW is summed slab by slab on a second
            # stream while its last contraction still runs
            import torch.distributed as dist
            if self.shards:
                self.shards.begin_step()
                self.B.spo_loss_fwd_bwd_scatter(*args, self.shards.table, entropy=self.entropy)
                dist.all_reduce(self.loss)
                self.shards.end_step()
                return
            self.B.spo_loss_fwd_bwd_slabs(*args, self.reducer.events, entropy=self.entropy)
            self.reducer.reduce(self.dW)
            dist.all_reduce(self.loss)
            self.reducer.finish()
            return
        self.B.spo_loss_fwd_bwd(*args, entropy=self.entropy)

    def loss_calls(self, h=None, y=None, logp_old=None, mask=None, cu=None):
        """The loss calls of one step on the chosen path."""
        if self.onepass:
            self.loss_onepass(h, y, logp_old, mask, cu)
        else:
            self.fwd(h, y, logp_old, mask, cu)
            self.bwd(h, y)

    def run(self):
        self.small()
        self.loss_calls()


def reduce_over_ranks(times_ms, tokens, world, device):
    """Replicas run independent mini-batches: the job's time is the slowest rank's (MAX of every
    timing), its work is the sum of the ranks' tokens (SUM).  Returns (times, tokens) on every rank."""
    import torch
    import torch.distributed as dist
    vals = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    toks = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
        dist.all_reduce(toks, op=dist.ReduceOp.SUM)
    return [float(x) for x in vals.tolist()], float(toks.item())


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    from paper_2509_13232_b200 import build as spo_build
    if rank == 0:
        spo_build.build()
    if world > 1:
        dist.barrier()
    dp_mode = args.parallelism == "dp" and dist.is_available() and dist.is_initialized()
    if dp_mode and (args.path != "onepass" or args.mask_frac > 0.0 or args.custom):
        raise SystemExit("--parallelism dp runs the one-pass loss on the unmasked named workloads")
    step = Step(args.workload, device, rank, args.responses, args.custom, args.mask_frac, args.path, args.entropy,
                dp_world=world if dp_mode else None, dw_slabs=args.dw_slabs, surrogate=args.surrogate,
                dual_clip=args.dual_clip, dw_reduce=args.dw_reduce)
    if args.surrogate == "gspo" and step.onepass:
        # a response's ratio needs all its tokens: spo_loss_fwd_bwd runs forward-then-backward for it
        step.flops_bwd = 6.0 * step.T * step.d * step.V
    peaks = read_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731  (timed on torch's current stream, which the library launches on)
    for _ in range(args.warmup):
        step.run()
    barrier()
    t_small = t_fwd = t_bwd = 0.0
    with ClockSampler(local_rank) as clocks:
        barrier()
        wall0 = time.perf_counter()
        marks = []
        for _ in range(args.steps):
            a, b, c, dd = ev(), ev(), ev(), ev()
            a.record(); step.small(); b.record()
            if step.onepass:
                c.record(); step.loss_onepass(); dd.record()        # no forward / backward boundary to time
            else:
                step.fwd(); c.record(); step.bwd(); dd.record()
            marks.append((a, b, c, dd))
        barrier()
        wall = time.perf_counter() - wall0
    total_ms = marks[0][0].elapsed_time(marks[-1][3])
    for a, b, c, dd in marks:
        t_small += a.elapsed_time(b); t_fwd += b.elapsed_time(c); t_bwd += c.elapsed_time(dd)
    status = int(step.status[0].item())

    # end to end: the step's inputs come from pinned host memory every step, the loss goes back
    D = step.data
    host = {k: D[k].cpu().pin_memory() for k in ("h", "y", "logp_old", "mask", "cu_seqlens")}
    host["rewards"] = step.rewards.cpu().pin_memory()
    host["uniforms"] = step.uniforms.cpu().pin_memory()
    names = ("h", "y", "logp_old", "mask", "cu_seqlens")
    # two sets of device input buffers: a copy stream fills one while the step runs on the other
    bufs = [{k: torch.empty_like(D[k]) for k in names} for _ in range(2)]
    small_bufs = [{"rewards": torch.empty_like(step.rewards), "uniforms": torch.empty_like(step.uniforms)}
                  for _ in range(2)]
    loss_host = torch.zeros(4, dtype=torch.float32).pin_memory()
    ids_host = torch.zeros(step.S, dtype=torch.int32).pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = loss_host.numel() * 4 + ids_host.numel() * 4
    main = torch.cuda.current_stream()
    copy_stream = torch.cuda.Stream(device=device)

    def e2e_run(n_steps):
        """n_steps whole steps, every one fed from pinned host memory; returns device milliseconds."""
        ready = [torch.cuda.Event() for _ in range(n_steps)]
        done = [torch.cuda.Event() for _ in range(n_steps)]
        s0, s1 = ev(), ev()
        s0.record(main)
        copy_stream.wait_event(s0)                      # the first copy starts inside the timed region
        for i in range(n_steps):
            b = i % 2
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(done[i - 2])  # the step that last used this buffer has finished
                for k in names:
                    bufs[b][k].copy_(host[k], non_blocking=True)
                small_bufs[b]["rewards"].copy_(host["rewards"], non_blocking=True)
                small_bufs[b]["uniforms"].copy_(host["uniforms"], non_blocking=True)
                ready[i].record(copy_stream)
            main.wait_event(ready[i])
            step.rewards, step.uniforms = small_bufs[b]["rewards"], small_bufs[b]["uniforms"]
            step.small()
            step.loss_calls(bufs[b]["h"], bufs[b]["y"], bufs[b]["logp_old"], bufs[b]["mask"], bufs[b]["cu_seqlens"])
            loss_host.copy_(step.loss, non_blocking=True)
            ids_host.copy_(step.ids, non_blocking=True)
            done[i].record(main)
        s1.record(main)
        torch.cuda.synchronize()
        return s0.elapsed_time(s1)

    e2e_steps = max(1, args.steps)
    e2e_run(1)
    barrier()
    e2e_ms = e2e_run(e2e_steps)
    barrier()

    (total_ms, e2e_ms, t_fwd, t_bwd, t_small), tokens_all = reduce_over_ranks(
        [total_ms, e2e_ms, t_fwd, t_bwd, t_small], step.n_tok, world, device)
    if rank != 0:
        return
    ms_per_step = total_ms / args.steps
    value = tokens_all / (ms_per_step / 1e3)
    gemm_ms = (t_fwd + t_bwd) / args.steps
    # tensor FLOPs of one rank's share over the slowest rank's time (per-GPU rate against a per-GPU peak)
    achieved = (step.flops_fwd + step.flops_bwd) / (gemm_ms / 1e3) / 1e12
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if dp_mode else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "custom" if args.custom else args.workload, "responses": step.S, "tokens": step.T, "d": step.d, "V": step.V,
                   "tracker_prompts": step.table_n, "l2": "inputs_exceed_l2", "loss_path": "onepass" if step.onepass else "split", "entropy_output": bool(args.entropy),
                   "surrogate": args.surrogate, "dual_clip": args.dual_clip,
                   "bwd_chunks": step.bwd_chunks, "mask_frac": step.mask_frac,
                   "parallelism": "dp%d" % world if dp_mode else ("replicas%d" % world if world > 1 else "single"),
                   "dw_reduce": args.dw_reduce if dp_mode else None},
        "gpu_launches": step.launches * args.steps,
        "device_status": status,
        "wall_s": wall,
        "breakdown_ms": ({"small": t_small / args.steps, "loss_fwd_bwd": t_bwd / args.steps} if step.onepass else
                         {"small": t_small / args.steps, "loss_fwd": t_fwd / args.steps, "loss_bwd": t_bwd / args.steps}),
        "roofline": {
            "bound": "tensor",
            "kernel": ("spo_gemm_kernel (E, DH, DW instantiations; all launches of a step; the duration is the whole "
                       "spo_loss_fwd_bwd call, which also holds the first-tile pass, the finalisation and the row-scaling kernels)" if step.onepass
                       else "spo_gemm_kernel (FWD, G, DH, DW instantiations; all launches of a step)"),
            "achieved": achieved, "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"],
            "peak_source": peaks["source"] + " sustained cuBLAS bf16",
            "frac_of_nominal_2250": achieved / 2250.0, "frac_of_burst": achieved / peaks["tflops_burst"],
            "flops_per_step": step.flops_fwd + step.flops_bwd,
            "flops_per_token": (step.flops_fwd + step.flops_bwd) / max(1, step.n_tok if step.mask_frac > 0.0 else step.T),
            "fwd_tflops": None if step.onepass else step.flops_fwd / (t_fwd / args.steps / 1e3) / 1e12,
            "bwd_tflops": None if step.onepass else step.flops_bwd / (t_bwd / args.steps / 1e3) / 1e12,
            # DRAM read+write bytes of all launches of one step (ncu counters of one chunk's launches, scaled by
            # token rows); known for the full cfg4 workload only.
            "traffic": CFG4_STEP_DRAM_BYTES.get("onepass" if step.onepass else "split") if (
                args.workload == "cfg4_8b_bf16" and not args.responses and not args.custom and not args.mask_frac) else None,
        },
        "e2e": {"value": tokens_all / (e2e_ms / e2e_steps / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "clocks": clocks.summary(),
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline_sample(args.workload, args.cpu_tokens)
    print(json.dumps(out), flush=True)


SMALL_SHAPES = {
    # workload: (table prompts N, batch B, uniforms M)
    "cfg2_tracker_scale": (1_000_000, 4096, 8192),
    "small_scaled": (1 << 28, 1 << 22, 8192),
    "small_scaled_26": (1 << 26, 1 << 22, 8192),      # a size that profiler captures with many passes can hold
    "small_scaled_24": (1 << 24, 1 << 20, 8192),
    "small_scaled_b24": (1 << 28, 1 << 24, 8192),     # the largest batch of the gather kernels
}


def run_small_kernels(args, local_rank):
    """Tracker / advantage / sampling kernels alone: time per call (CUDA events, L2 flushed by writing a
    512 MB buffer before every timed call) and achieved algorithmic GB/s against the measured HBM copy rate."""
    import torch
    from paper_2509_13232_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    N, Bn, M = SMALL_SHAPES[args.workload]
    peaks = read_peaks()
    g = torch.Generator(device=dev)
    g.manual_seed(20250913)
    ab = torch.rand((N, 2), generator=g, device=dev) * 12 + 0.1
    v0 = torch.rand(N, generator=g, device=dev)
    u = torch.rand(M, generator=g, device=dev).clamp_(0, 0.999999)
    ids = torch.randperm(N, generator=g, device=dev)[:Bn].to(torch.int32)
    r = (torch.rand(Bn, generator=g, device=dev) < 0.4).float()
    kl = torch.rand(Bn, generator=g, device=dev) * 0.05
    n_draw = min(4096, Bn)
    out_ids = torch.empty(n_draw, dtype=torch.int32, device=dev)
    a_norm = torch.empty(Bn, device=dev)
    stats = torch.empty(8, device=dev)
    st = torch.zeros(4, dtype=torch.int32, device=dev)
    ws = torch.empty(B.spo_workspace_bytes(B.WS_SAMPLE, N=N, M=M), dtype=torch.uint8, device=dev)
    wsa = torch.empty(B.spo_workspace_bytes(B.WS_ADVANTAGES, B=Bn), dtype=torch.uint8, device=dev)
    ab2 = torch.empty_like(ab)
    p = B.default_params()
    flush = torch.empty(128 * 1024 * 1024, dtype=torch.float32, device=dev)
    calls = {
        "spo_tracker_init": (lambda: B.spo_tracker_init(ab2, v0, p), 12 * N, 1),
        # launches: sums, prefix, search, accept for tables of up to 2^20 prompts; sums, search, accept above
        "spo_sample_prompts": (lambda: B.spo_sample_prompts(ab, u, n_draw, out_ids, None, ws, p, st), 8 * N,
                               4 if N <= (1 << 20) else 3),
        "spo_advantages": (lambda: B.spo_advantages(ab, ids, r, None, a_norm, stats, wsa, p, st), 28 * Bn,
                           1 if Bn <= 8192 else 2),
        "spo_tracker_update": (lambda: B.spo_tracker_update(ab, ids, r, kl, 0, p, st), 28 * Bn, 1),
        # advantage + update in one pass over the entries: per element 4 B id, 4 B reward, 4 B divergence,
        # 8 B entry read and written back, 4 B advantage written, read and written normalised = 36 B
        "spo_advantages_update": (lambda: B.spo_advantages_update(ab, ids, r, kl, 0, None, a_norm, stats, wsa, p, st),
                                  36 * Bn, 1 if Bn <= 8192 else 2),
    }
    # What a random 8-byte read-modify-write costs the memory system: the entry comes in as a 64-byte
    # DRAM burst (two 32-byte sectors) and its dirty 32-byte sector goes back later; the streamed arrays
    # cost their own bytes.  Time of that traffic at the measured copy rate = the bound for the gathers.
    gather_bound_bytes = {"spo_advantages": (64 + 20) * Bn, "spo_tracker_update": (64 + 32 + 12) * Bn,
                          "spo_advantages_update": (64 + 32 + 28) * Bn}
    out_calls, total_ms, total_bytes, launches = {}, 0.0, 0, 0
    with ClockSampler(local_rank) as clocks:
        for name, (fn, nbytes, n_launch) in calls.items():
            ts = []
            for i in range(args.warmup + args.steps):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record()
                torch.cuda.synchronize()
                if i >= args.warmup:
                    ts.append(e0.elapsed_time(e1))
            ts.sort()
            ms = ts[len(ts) // 2]
            # the same call replayed from a CUDA graph: what the device needs for it once the host's launch
            # calls (four per sampling call) are out of the way -- at the paper's sizes they are most of `ms`
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                fn()
            tg = []
            for i in range(args.warmup + args.steps):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); graph.replay(); e1.record()
                torch.cuda.synchronize()
                if i >= args.warmup:
                    tg.append(e0.elapsed_time(e1))
            tg.sort()
            out_calls[name] = {"ms": ms, "graph_ms": tg[len(tg) // 2], "algorithmic_bytes": nbytes,
                               "GB/s": nbytes / ms / 1e6, "frac_of_hbm": nbytes / ms / 1e6 / peaks["hbm_gbs"]}
            if name in gather_bound_bytes:
                bound_ms = gather_bound_bytes[name] / peaks["hbm_gbs"] / 1e6
                out_calls[name].update({"random_access_bound_ms": bound_ms, "frac_of_random_access_bound": bound_ms / ms})
            if name not in ("spo_advantages", "spo_tracker_update"):       # the fused call does their work in the step
                total_ms += ms
                total_bytes += nbytes
            launches += n_launch * args.steps
    # reference for the gathers: the same random 8-byte rows fetched by a library primitive
    idx64 = ids.to(torch.int64)
    picked = torch.empty((Bn, 2), device=dev)
    tr = []
    for i in range(args.warmup + args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); torch.index_select(ab, 0, idx64, out=picked); e1.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            tr.append(e0.elapsed_time(e1))
    tr.sort()
    gather_ref_ms = tr[len(tr) // 2]
    dom = out_calls["spo_sample_prompts"]
    print(json.dumps({
        "metric": "tracker / advantage / sampling kernels, achieved HBM GB/s (algorithmic bytes)",
        "value": total_bytes / total_ms / 1e6, "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": args.workload, "N": N, "B": Bn, "M": M, "l2": "flushed_before_each_call"},
        "gpu_launches": launches, "device_status": int(st[0].item()), "calls": out_calls,
        "random_gather_reference": {"what": "torch.index_select of the same B random 8-byte table rows", "ms": gather_ref_ms,
                                    "accesses_per_s": Bn / gather_ref_ms * 1e3},
        "roofline": {"bound": "hbm", "kernel": "sample_tile_sums_kernel (within spo_sample_prompts)",
                     "achieved": dom["GB/s"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": dom["frac_of_hbm"],
                     "peak_source": peaks["source"] + " copy", "traffic": None},
        "clocks": clocks.summary(),
    }), flush=True)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


ORACLE_ROWS = 512      # token rows of the CPU-oracle sample (both the cpu_baseline leg and --impl reference)


def oracle_sample(workload, n_rows):
    """The bounded sample both CPU legs time: n_rows synthetic token rows of the workload's shape
    (H ~ N(0,1), W ~ N(0, w_std), bf16-rounded, targets uniform), W widened to float64 once, here,
    outside every timed region."""
    from paper_2509_13232_b200 import inputs
    d, V, w_std, _, _ = LOSS_SHAPES[workload]
    rng = inputs.rng_for(int(workload[3]), 9)
    h = inputs.round_to_bf16(rng.standard_normal((n_rows, d)).astype(np.float32)).astype(np.float64)
    w = inputs.round_to_bf16((rng.standard_normal((V, d)) * w_std).astype(np.float32)).astype(np.float64)
    y = rng.integers(0, V, n_rows).astype(np.int32)
    lo = np.full(n_rows, -np.log(V), dtype=np.float32)
    a_tok = np.full(n_rows, 0.5, dtype=np.float32)
    text = ("oracle loss forward+backward on %d synthetic token rows at full d=%d, V=%d (numpy float64, W widened "
            "once outside the timed region); the tracker/sampling steps are negligible beside it" % (n_rows, d, V))
    return (h, w, y, lo, a_tok), text


def oracle_slice_seconds(h, w, y, logp_old, a_tok):
    """Time the oracle, as it stands, on the given token rows (forward + backward)."""
    from oracle import spo_oracle as O
    n_rows = h.shape[0]
    cu = np.arange(n_rows + 1)
    t0 = time.perf_counter()
    fwd = O.loss_forward(h, w, y, logp_old, None, cu, a_tok)
    O.loss_backward(h, w, y, fwd["lse"], fwd["coef"], 1.0)
    return time.perf_counter() - t0


def cpu_baseline_sample(workload, n_rows):
    sample, text = oracle_sample(workload, n_rows)
    sec = oracle_slice_seconds(*sample)
    return {"value": n_rows / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": text,
            "seconds": sec}


def run_reference(args, rank, world):
    """The reference arm: the float64 CPU oracle on the same bounded sample per step (rank 0 only)."""
    if rank != 0:
        return
    d, V = LOSS_SHAPES[args.workload][:2]
    n_rows = args.cpu_tokens
    sample, text = oracle_sample(args.workload, n_rows)
    for _ in range(args.warmup):
        oracle_slice_seconds(*sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_slice_seconds(*sample)
    sec = (time.perf_counter() - t0) / args.steps
    value = n_rows / sec
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "tokens": n_rows, "d": d, "V": V},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": "each step = " + text},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


def spawn_ranks(n):
    """`python bench.py --gpus N` without a launcher: start N copies of this command, one per GPU, with
    the rendezvous environment a launcher would give them (127.0.0.1, a free port).  Rank 0 prints the
    JSON line.  Returns the worst exit code."""
    import socket
    if "--rehearse-host" not in sys.argv:
        import torch
        have = torch.cuda.device_count()
        if have < n:
            sys.stderr.write("bench.py: --gpus %d asked for, %d CUDA device(s) visible\n" % (n, have))
            return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")              # the communicator log (transport, NVLS) goes to stderr
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    # a rank that dies would leave the others waiting in a collective: stop them when one fails
    codes = [None] * n
    while any(c is None for c in codes):
        for i, pr in enumerate(procs):
            if codes[i] is None:
                codes[i] = pr.poll()
        if any(c not in (None, 0) for c in codes):
            for i, pr in enumerate(procs):
                if codes[i] is None:
                    pr.terminate()
                    codes[i] = pr.wait()
            break
        time.sleep(0.2)
    return max(abs(c) for c in codes)


def rehearse_host(args, rank, world):
    """The host side of a multi-rank run without any GPU: rendezvous over gloo, the token-balanced split
    of the mini-batch, the dW slab plan, the reduction of timings and token counts, and the merge of
    per-rank advantage statistics -- on dummy values.  Rank 0 prints the plan as one JSON line."""
    import torch
    import torch.distributed as dist
    from paper_2509_13232_b200 import binding as B
    from paper_2509_13232_b200 import dp, inputs
    if world > 1:
        dist.init_process_group("gloo")
    try:
        d, V = LOSS_SHAPES[args.workload][:2]
        lengths = inputs.workload_lengths(args.workload)
        if args.responses:
            lengths = lengths[:args.responses]
        parts = dp.partition_by_tokens(lengths, world)
        mine = int(np.sum(np.asarray(lengths)[parts[rank]])) if parts[rank] else 0
        times, tokens_all = reduce_over_ranks([100.0 + rank, 50.0 - rank], mine, world, torch.device("cpu"))
        n_tok, n_resp = dp.global_counts(mine, len(parts[rank]))
        rec = torch.tensor([float(rank), 1.0, float(len(parts[rank])), 2.0 * len(parts[rank]), 0, 0, 0, 0])
        mu, sigma = dp.global_advantage_stats(rec)
        slabs = B.spo_dw_slab_rows(V, d, args.dw_slabs)
        if rank == 0:
            print(json.dumps({"rehearsal": True, "n_ranks": world, "parallelism": args.parallelism,
                              "tokens_per_rank": [int(np.sum(np.asarray(lengths)[p])) for p in parts],
                              "responses_per_rank": [len(p) for p in parts], "tokens_all": tokens_all,
                              "global_tokens": n_tok, "global_responses": n_resp, "max_times": times,
                              "merged_mu_sigma": [mu, sigma], "dw_slab_rows": slabs,
                              "dw_slab_order": dp.slab_schedule(slabs)}), flush=True)
    finally:
        if world > 1:
            dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4_8b_bf16", choices=sorted(LOSS_SHAPES) + sorted(SMALL_SHAPES))
    ap.add_argument("--cpu-tokens", type=int, default=None, help="token rows of the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--custom", type=lambda v: tuple(int(x) for x in v.split(",")), default=None,
                    help="T,d,V: time the loss path on another LM-head shape (eight equal responses)")
    ap.add_argument("--mask-frac", type=float, default=0.0,
                    help="mask this share of the tokens in contiguous spans and run the loss over the unmasked rows "
                         "only (spo_loss_fwd_bwd_rows; with --path split: the backward over the rows with gradient, "
                         "spo_loss_bwd_rows)")
    ap.add_argument("--path", default="onepass", choices=["onepass", "split"],
                    help="loss as one spo_loss_fwd_bwd call (default) or as spo_loss_fwd + spo_loss_bwd")
    ap.add_argument("--surrogate", default="ppo_clip", choices=["ppo_clip", "cispo", "gspo"],
                    help="objective of the loss calls: the paper's PPO-Clip, or one of the two it names as compatible")
    ap.add_argument("--dual-clip", type=float, default=0.0, help="second clip for negative advantages (0 = off)")
    ap.add_argument("--entropy", action="store_true", help="also ask the loss call for the per-token policy entropy")
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "dp"],
                    help="with more than one GPU: every rank its own mini-batch (weak scaling, no data-path "
                         "collective), or ONE mini-batch split over the ranks by token count with dW summed over the "
                         "ranks, overlapped slab by slab with its last contraction (strong scaling)")
    ap.add_argument("--dw-slabs", type=int, default=8, help="slabs the last dW contraction is cut into (dp)")
    ap.add_argument("--dw-reduce", choices=["allreduce", "scatter"], default="allreduce",
                    help="dp: sum dW over the ranks with all-reduces per slab behind the last contraction (default), "
                         "or have that contraction add its tiles into per-rank vocabulary shards in peer-mapped "
                         "memory (spo_loss_fwd_bwd_scatter; every rank ends with its rows of dW)")
    ap.add_argument("--rehearse-host", action="store_true",
                    help="no GPU work: start the ranks (gloo), plan the data-parallel split and the dW slabs, run the "
                         "host-side exchanges on dummy values and print the plan (used by the CPU tests)")
    ap.add_argument("--responses", type=int, default=None,
                    help="use only the first S responses of the workload (small cases for profiling)")
    args = ap.parse_args()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.workload in LOSS_SHAPES and (
            args.impl == "ours" or args.rehearse_host):
        sys.exit(spawn_ranks(args.gpus))          # one process per GPU, as a launcher would start them
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.rehearse_host:
        rehearse_host(args, rank, world)
        return
    if args.workload in SMALL_SHAPES:
        if rank == 0:
            run_small_kernels(args, local_rank)
        return
    if args.cpu_tokens is None:
        args.cpu_tokens = ORACLE_ROWS
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    # a process group for N > 1 ranks, and for one rank under a launcher when the data-parallel step is asked
    # for (its exchanges are then the identity: what that step costs by itself on one GPU)
    grouped = world > 1 or (args.parallelism == "dp" and "WORLD_SIZE" in os.environ)
    if grouped:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if grouped:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
