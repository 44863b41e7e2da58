"""Host-side glue for data-parallel training over responses (one process per GPU).

Each rank holds its share of the mini-batch's responses and the replicated W and tracker table.
Three small exchanges make the ranks' results those of the whole mini-batch:

  1. advantage statistics: every rank calls spo_advantages for its raw advantages and
     (mu, sigma, B, M2, near-zero counts); `global_advantage_stats` gathers the 32-byte records, merges them and
     returns the mini-batch mu and sigma for spo_advantages_apply;
  2. denominators of the objective: `global_counts` sums the ranks' unmasked-token and active-
     response counts; they go into spo_params.global_tokens / global_responses;
  3. after spo_loss_bwd: `allreduce_sum` on dW (and on the scalar loss); dH rows are already final.

Only torch.distributed calls and a few lines of float64 arithmetic live here; nothing of the
path itself.
"""

from __future__ import annotations

import math


def merge_moments(parts):
    """Merge (mean, M2, count) records, M2 = sum of squared deviations from the record's own mean
    (pairwise update of Chan et al.).  Returns (mean, M2, count)."""
    mean, m2, n = 0.0, 0.0, 0.0
    for mu_b, m2_b, n_b in parts:
        mu_b, m2_b, n_b = float(mu_b), float(m2_b), float(n_b)
        if n_b <= 0:
            continue
        tot = n + n_b
        delta = mu_b - mean
        mean += delta * n_b / tot
        m2 += m2_b + delta * delta * n * n_b / tot
        n = tot
    return mean, m2, n


def sigma_from(m2, n, ddof=0):
    den = n - ddof
    return math.sqrt(m2 / den) if den > 0 else 0.0


def global_advantage_stats(stats, ddof=0, group=None):
    """`stats` is this rank's [8] tensor (mu, sigma, B, M2, n_lo, n_hi, 0, 0) from spo_advantages.  Returns the
    mini-batch (mu, sigma) as Python floats, identical on every rank."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        rows = [stats.detach().cpu().double()]
    else:
        bucket = [torch.empty_like(stats) for _ in range(world)]
        dist.all_gather(bucket, stats.contiguous(), group=group)
        rows = [b.detach().cpu().double() for b in bucket]
    mean, m2, n = merge_moments([(float(r[0]), float(r[3]), float(r[2])) for r in rows])
    return mean, sigma_from(m2, n, ddof)


def global_counts(n_tokens, n_responses, device=None, group=None):
    """Sum of the ranks' unmasked-token and active-response counts."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([int(n_tokens), int(n_responses)], dtype=torch.int64, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return int(t[0].item()), int(t[1].item())


def allreduce_sum(tensor, group=None):
    """In-place sum over ranks (dW, the scalar loss)."""
    import torch.distributed as dist
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(tensor, op=dist.ReduceOp.SUM, group=group)
    return tensor


def partition_by_tokens(lengths, world):
    """Responses of one mini-batch dealt to `world` ranks so that the ranks' token counts are as even
    as a greedy pass makes them: longest response first, each to the rank that holds the fewest tokens
    so far (ties: lowest rank).  Returns one ascending list of response indices per rank; every rank
    computes the same partition from the same lengths."""
    order = sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i))
    load = [0] * world
    parts = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        parts[r].append(i)
        load[r] += int(lengths[i])
    return [sorted(p) for p in parts]


def slab_schedule(row_begin):
    """(slab index, first row, end row) in the order the slabs of dW become final."""
    return [(k, int(row_begin[k]), int(row_begin[k + 1])) for k in range(len(row_begin) - 1)]


class SlabAllReduce:
    """Sums dW over the ranks slab by slab while its last contraction still runs.

    spo_loss_fwd_bwd_slabs records events[k] on the compute stream once rows row_begin[k] ..
    row_begin[k+1]-1 of dW are final.  `reduce` makes a second stream wait for each event in turn and
    issues the all-reduce of that slab there, so the transfer of slab k overlaps the contraction of
    slab k+1; `finish` makes the compute stream wait for the last reduction.  Only torch.distributed
    collectives are used (NCCL on GPUs); no kernel of the library reads another rank's memory.
    """

    def __init__(self, row_begin, device, group=None):
        import torch
        self.row_begin = [int(x) for x in row_begin]
        self.group = group
        self.stream = torch.cuda.Stream(device=device)
        self.events = []
        for _ in range(len(self.row_begin) - 1):
            ev = torch.cuda.Event(enable_timing=False)
            ev.record()                    # a torch event owns its CUDA event only after its first record
            self.events.append(ev)
        self.done = torch.cuda.Event(enable_timing=False)
        self.works = []

    def reduce(self, dW):
        import torch
        import torch.distributed as dist
        self.works = []
        with torch.cuda.stream(self.stream):
            for k, lo, hi in slab_schedule(self.row_begin):
                self.stream.wait_event(self.events[k])
                if dist.is_initialized() and dist.get_world_size(self.group) > 1:
                    self.works.append(dist.all_reduce(dW[lo:hi], op=dist.ReduceOp.SUM, group=self.group, async_op=True))
            for w in self.works:
                w.wait()                   # stream-level wait: the side stream orders behind the collectives
            self.done.record(self.stream)

    def finish(self):
        import torch
        torch.cuda.current_stream().wait_event(self.done)


class PeerShards:
    """Vocabulary-row shards of dW, one per rank, that every rank can write: the target of
    spo_loss_fwd_bwd_scatter.  Each rank owns an fp32 [rows_per_shard][d] buffer in memory that is mapped
    into all ranks of the group (torch's symmetric memory); `table` is the shard table for the call.

        shards.begin_step()      # zero this rank's shard; all ranks' zeroing is visible before anyone adds
        binding.spo_loss_fwd_bwd_scatter(..., shards.table)
        shards.end_step()        # every rank's additions have landed: shards.local holds this rank's rows of dW

    The exchange itself is the library's: store-reductions into the owners' memory from the epilogue of the
    last dW contraction (over NVLink for a peer's shard).  Not run on more than one GPU so far.
    """

    def __init__(self, V, d, device, group=None):
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem
        from . import binding
        group = group if group is not None else dist.group.WORLD
        world = dist.get_world_size(group)
        self.rows_per_shard = -(-int(V) // world)
        self.local = symm_mem.empty((self.rows_per_shard, int(d)), dtype=torch.float32, device=device)
        self.handle = symm_mem.rendezvous(self.local, group)
        self.table = binding.dw_shards([int(p) for p in self.handle.buffer_ptrs], self.rows_per_shard)

    def begin_step(self):
        self.local.zero_()
        self.handle.barrier()

    def end_step(self):
        self.handle.barrier()
