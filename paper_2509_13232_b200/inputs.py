"""Seeded synthetic inputs for the SPO hot path.

This module only draws random numbers and shapes them; it contains none of the
method's arithmetic (no tracker, advantage, surrogate or gradient formulas).
Both the CUDA path and the CPU oracle are fed from here, so the two sides see
the same stored values.  Where a recipe is phrased relative to the model's own
outputs ("targets sampled from the model softmax", "old log-probs = new
log-probs + noise"), the logits are formed here with one library matmul and
the target is the argmax of logits plus Gumbel noise; the base log-prob is a
library log-softmax.  These only shape plausible inputs.

The workloads stand in for the paper's Qwen3-8B tool-integrated-reasoning
runs (appendix "Training and Evaluation Details": prompt batch 2048 in
mini-batches of 256, responses up to 16384 tokens), whose weights and data are
not available: the LM-head shape (d, V), the packed variable-length responses
and the binary rewards are kept, the values are random.
"""

from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20250913


def seed_for(cfg: int, stream: int) -> int:
    return BASE_SEED + 1000 * int(cfg) + int(stream)


def rng_for(cfg: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed_for(cfg, stream)))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    bits = (bits + 0x7FFF + lsb) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).reshape(x.shape)


# -------------------------------------------------------------------------
# response lengths
# -------------------------------------------------------------------------

def lengths_uniform(rng, n_seq, lo, hi):
    return rng.integers(lo, hi + 1, size=n_seq).astype(np.int64)


def lengths_lognormal(rng, n_seq, mean_tokens, sigma, lo, hi):
    mu = np.log(mean_tokens) - 0.5 * sigma * sigma
    raw = np.rint(rng.lognormal(mu, sigma, size=n_seq))
    return np.clip(raw, lo, hi).astype(np.int64)


def lengths_pareto(rng, n_seq, x_m, alpha, lo, hi):
    u = 1.0 - rng.random(n_seq)          # in (0, 1]
    raw = np.rint(x_m * u ** (-1.0 / alpha))
    return np.clip(raw, lo, hi).astype(np.int64)


def cu_seqlens_from(lengths) -> np.ndarray:
    cu = np.zeros(len(lengths) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lengths)
    return cu


# -------------------------------------------------------------------------
# tracker table, batch, uniforms
# -------------------------------------------------------------------------

@dataclass
class TrackerBatch:
    ab: np.ndarray            # [N, 2] fp32 interleaved (alpha, beta)
    kl_table: np.ndarray      # [N] fp32 per-prompt divergence
    ids: np.ndarray           # [B] int32 distinct
    rewards: np.ndarray       # [B] fp32 in {0, 1}
    kl: np.ndarray            # [B] fp32 = kl_table[ids]
    uniforms: np.ndarray      # [M] fp32 in [0, 1)
    v0: np.ndarray | None = None   # [N] fp32 initial estimates when built by Algorithm 2


def uniforms_f32(rng, m):
    """fp32 uniforms in [0,1) with 24 random bits each (exactly representable)."""
    return (rng.integers(0, 1 << 24, size=m).astype(np.float32) / np.float32(1 << 24)).astype(np.float32)


def tracker_table_equilibrium(rng, n):
    """Estimates ~ Beta(2,2) with effective sample size alpha+beta ~ U[8,25]."""
    v = rng.beta(2.0, 2.0, size=n)
    neff = rng.uniform(8.0, 25.0, size=n)
    ab = np.empty((n, 2), dtype=np.float32)
    ab[:, 0] = (v * neff).astype(np.float32)
    ab[:, 1] = ((1.0 - v) * neff).astype(np.float32)
    return ab, v


def tracker_batch(cfg, n, b, m, table="equilibrium", reward_p=None):
    """Table of n prompts, b distinct batch ids, rewards, divergences, m uniforms.

    table="equilibrium": estimates ~ Beta(2,2), alpha+beta ~ U[8,25].
    table="init8": v0 = k/8 with k ~ Binomial(8, 0.5); ab is left for the
    caller to build with Algorithm 2 from ``v0`` (ab holds zeros).
    Rewards ~ Bernoulli(reward_p) if given, else Bernoulli(estimate of the id).
    """
    rng = rng_for(cfg, 1)
    v0 = None
    if table == "equilibrium":
        ab, est = tracker_table_equilibrium(rng, n)
    elif table == "init8":
        v0 = (rng.binomial(8, 0.5, size=n) / 8.0).astype(np.float32)
        ab = np.zeros((n, 2), dtype=np.float32)
        est = v0.astype(np.float64)
    else:
        raise ValueError(table)
    kl_table = rng.lognormal(-4.0, 1.0, size=n).astype(np.float32)
    ids = rng.permutation(n)[:b].astype(np.int32)
    p = est[ids] if reward_p is None else np.full(b, float(reward_p))
    rewards = (rng.random(b) < p).astype(np.float32)
    uniforms = uniforms_f32(rng, m)
    return TrackerBatch(ab=ab, kl_table=kl_table, ids=ids, rewards=rewards,
                        kl=kl_table[ids].copy(), uniforms=uniforms, v0=v0)


# -------------------------------------------------------------------------
# loss inputs (host / numpy path: sizes the oracle can finish)
# -------------------------------------------------------------------------

@dataclass
class LossBatch:
    h: np.ndarray             # [T, d] fp32 (bf16-representable when bf16=True)
    w: np.ndarray             # [V, d] fp32 (bf16-representable when bf16=True)
    y: np.ndarray             # [T] int32
    logp_old: np.ndarray      # [T] fp32
    mask: np.ndarray          # [T] uint8
    cu_seqlens: np.ndarray    # [S+1] int32
    a_norm: np.ndarray        # [S] fp32
    bf16: bool = False
    meta: dict = field(default_factory=dict)


def _log_softmax_rows(z):
    from scipy.special import log_softmax
    return log_softmax(z, axis=1)


def loss_batch(cfg, lengths, d, v, w_std, bf16, old_noise, target="softmax",
               mask_p=None, a_norm=None):
    """Packed loss inputs on the host.

    h ~ N(0,1), w ~ N(0,w_std); target="uniform": y ~ U{0..V-1};
    target="softmax": y = argmax(logits + Gumbel) (a draw from softmax(logits));
    logp_old = log_softmax(logits)[y] + N(0, old_noise);
    mask: all ones, or Bernoulli(mask_p) zeros sprinkled in;
    a_norm: given, or N(0,1) draws as a stand-in for normalised advantages.
    """
    rng = rng_for(cfg, 2)
    lengths = np.asarray(lengths, dtype=np.int64)
    t = int(lengths.sum())
    h = rng.standard_normal((t, d)).astype(np.float32)
    w = (rng.standard_normal((v, d)) * w_std).astype(np.float32)
    if bf16:
        h = round_to_bf16(h)
        w = round_to_bf16(w)
    z = h.astype(np.float64) @ w.astype(np.float64).T
    if target == "uniform":
        y = rng.integers(0, v, size=t).astype(np.int32)
    elif target == "softmax":
        gumbel = -np.log(-np.log(rng.random((t, v))))
        y = np.argmax(z + gumbel, axis=1).astype(np.int32)
    else:
        raise ValueError(target)
    base = _log_softmax_rows(z)[np.arange(t), y] if t else np.zeros(0)
    logp_old = (base + rng.normal(0.0, old_noise, size=t)).astype(np.float32)
    if mask_p is None:
        mask = np.ones(t, dtype=np.uint8)
    else:
        mask = (rng.random(t) >= mask_p).astype(np.uint8)
    if a_norm is None:
        a_norm = rng.standard_normal(len(lengths)).astype(np.float32)
    return LossBatch(h=h, w=w, y=y, logp_old=logp_old, mask=mask,
                     cu_seqlens=cu_seqlens_from(lengths),
                     a_norm=np.asarray(a_norm, dtype=np.float32), bf16=bf16,
                     meta={"cfg": cfg, "T": t, "d": d, "V": v, "S": len(lengths)})


# -------------------------------------------------------------------------
# the five named workloads (shapes and distributions)
# -------------------------------------------------------------------------

WORKLOADS = {
    # name: description of the recipe (shapes; distributions are in the builders below)
    "cfg1_tiny_fp32": dict(S=16, d=64, V=512, N=16, B=16, M=64),
    "cfg2_tracker_scale": dict(N=1_000_000, B=4096, M=8192),
    "cfg3_small_bf16": dict(S=64, d=1024, V=151936),
    "cfg4_8b_bf16": dict(S=128, d=4096, V=151936),
    "cfg5_longtail_bf16": dict(S=32, d=4096, V=151936, N=100_000, B=4096, M=8192),
}


def workload_lengths(name):
    """Response lengths of a named workload (seeded)."""
    if name == "cfg1_tiny_fp32":
        return lengths_uniform(rng_for(1, 0), 16, 8, 32)
    if name == "cfg3_small_bf16":
        return lengths_uniform(rng_for(3, 0), 64, 256, 2048)
    if name == "cfg4_8b_bf16":
        # sigma is not fixed by the workload statement; 0.5 keeps the clipped mean near 2048
        return lengths_lognormal(rng_for(4, 0), 128, 2048.0, 0.5, 64, 8192)
    if name == "cfg5_longtail_bf16":
        # x_m = 3300 gives about 250k tokens in total after clipping to [512, 32768]
        return lengths_pareto(rng_for(5, 0), 32, 3300.0, 1.5, 512, 32768)
    raise ValueError(name)


def cfg1_tiny():
    """Tiny fp32 step: loss inputs plus a 16-prompt tracker built by Algorithm 2."""
    lengths = workload_lengths("cfg1_tiny_fp32")
    tb = tracker_batch(1, 16, 16, 64, table="init8", reward_p=0.5)
    lb = loss_batch(1, lengths, 64, 512, 0.05, False, 0.05, target="uniform", a_norm=np.zeros(16))
    return tb, lb


# -------------------------------------------------------------------------
# device-side generation for sizes the host cannot hold comfortably
# -------------------------------------------------------------------------

def loss_batch_device(cfg, lengths, d, v, w_std, old_noise, device, adv_p=0.3, t_chunk=2048, w_cfg=None):
    """bf16 loss inputs generated on ``device`` with a seeded torch generator.

    ``w_cfg`` seeds W by itself (default: ``cfg``): data-parallel ranks draw their own responses
    (different ``cfg``) against the same replicated W (same ``w_cfg``).

    Returns a dict of torch tensors: h [T,d] bf16, w [V,d] bf16, y [T] int32,
    logp_old [T] fp32, mask [T] uint8, cu_seqlens [S+1] int32 and rewards [S]
    fp32 ~ Bernoulli(adv_p).  Targets are Gumbel-max draws from chunked
    library-matmul logits; logp_old is the library log-softmax at the target
    plus N(0, old_noise).
    """
    import torch
    lengths = np.asarray(lengths, dtype=np.int64)
    t = int(lengths.sum())
    g = torch.Generator(device=device)
    g.manual_seed(seed_for(cfg, 3))
    h = torch.randn((t, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    gw = torch.Generator(device=device)
    gw.manual_seed(seed_for(cfg if w_cfg is None else w_cfg, 6))
    w = (torch.randn((v, d), generator=gw, device=device, dtype=torch.float32) * w_std).to(torch.bfloat16)
    y = torch.empty(t, dtype=torch.int32, device=device)
    logp_old = torch.empty(t, dtype=torch.float32, device=device)
    for t0 in range(0, t, t_chunk):
        z = (h[t0:t0 + t_chunk] @ w.T).float()
        u = torch.rand(z.shape, generator=g, device=device, dtype=torch.float32).clamp_(1e-20, 1.0)
        yy = torch.argmax(z - torch.log(-torch.log(u)), dim=1)
        base = torch.log_softmax(z, dim=1).gather(1, yy[:, None])[:, 0]
        noise = torch.randn(base.shape, generator=g, device=device, dtype=torch.float32) * old_noise
        y[t0:t0 + t_chunk] = yy.to(torch.int32)
        logp_old[t0:t0 + t_chunk] = base + noise
        del z, u
    rng = rng_for(cfg, 4)
    rewards = torch.from_numpy((rng.random(len(lengths)) < adv_p).astype(np.float32)).to(device)
    return {
        "h": h, "w": w, "y": y, "logp_old": logp_old,
        "mask": torch.ones(t, dtype=torch.uint8, device=device),
        "cu_seqlens": torch.from_numpy(cu_seqlens_from(lengths)).to(device),
        "rewards": rewards, "T": t, "d": d, "V": v, "S": len(lengths),
    }
