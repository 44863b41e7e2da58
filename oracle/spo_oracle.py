"""Float64 CPU oracle for the SPO (Single-stream Policy Optimization) hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of what
the paper defines; the CUDA library is checked against it.  It shares no code
with the CUDA path, imports nothing from it, and must never be called from the
product path (only from tests, the smoke check and the CPU-baseline leg of the
benchmark).

Everything is numpy float64.  Where floating point decides an integer (the
sampled prompt ids) the decision itself is taken on integers: the selector
(``sample_prompts``) receives the fp32 sampling weights as an input and
quantises them exactly, so "bit-exact ids given the same uniforms and weights"
needs no floating-point agreement beyond the weights themselves, which are
checked against ``sampling_weights`` (the float64 definition) separately.

Pinned by tests/test_oracle_pins.py against closed forms, brute force, finite
differences and the constants the paper prints.  Pieces whose parameters the
paper never gives a value or a formula for (``d_half``; the two objectives
Sec. 3.2 only names, ``SUR_CISPO`` and ``SUR_GSPO``; the optional second clip
``dual_clip``, which is not in the paper at all; the whole-step
composition, for which no worked example is printed) are "parity unpinned" by
the paper itself and are pinned only through the identities listed in that
test file.

Paper sections: Sec. 3.1 (KL-adaptive value tracker), Sec. 3.2 (advantage,
global normalisation, PPO-Clip objective), Sec. 3.3 and Eq. "sampling_coef"
(prioritised sampling), Algorithm 1 (training loop), Algorithm 2
(initialisation), appendix "Training and Evaluation Details" (constants).
"""

from __future__ import annotations

import numpy as np

# Constants printed in the appendix "Training and Evaluation Details" and Sec. 3.3.
RHO_MIN = 0.875
RHO_MAX = 0.96
EPS_EXPLORE = 0.05
CLIP_LO = 0.2
CLIP_HI = 0.28
N0_SAMPLES = 8


# --------------------------------------------------------------------------
# Sec. 3.1 -- value tracker
# --------------------------------------------------------------------------

def tracker_init(v0, rho_min=RHO_MIN):
    """Algorithm 2: N0 = 1/(1-rho_min); alpha0 = N0*v0; beta0 = N0*(1-v0)."""
    v0 = np.asarray(v0, dtype=np.float64)
    n0 = 1.0 / (1.0 - float(rho_min))
    return n0 * v0, n0 * (1.0 - v0)


def value_estimate(alpha, beta):
    """Posterior mean v = alpha/(alpha+beta) (Sec. 3.1).

    The paper does not say what an empty tracker (alpha+beta = 0) estimates;
    the reading taken is the uninformed 0.5.
    """
    alpha = np.asarray(alpha, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    n = alpha + beta
    safe = np.where(n > 0.0, n, 1.0)
    return np.where(n > 0.0, alpha / safe, 0.5)


def forgetting_factor(kl, d_half, rho_min=RHO_MIN, rho_max=RHO_MAX):
    """rho = 2^(-D/D_half), kept inside [rho_min, rho_max] by a hard clamp (Sec. 3.1)."""
    kl = np.asarray(kl, dtype=np.float64)
    rho = np.exp2(-kl / float(d_half))
    return np.minimum(np.maximum(rho, float(rho_min)), float(rho_max))


def tracker_update(alpha, beta, ids, r, kl, d_half, rho_min=RHO_MIN, rho_max=RHO_MAX):
    """Tracker update equation of Sec. 3.1, applied to the batch entries in order.

    alpha <- rho*alpha + r ; beta <- rho*beta + (1-r), at table row ids[j].
    ``kl`` holds one divergence per batch entry.  Returns new copies.
    """
    alpha = np.array(alpha, dtype=np.float64, copy=True)
    beta = np.array(beta, dtype=np.float64, copy=True)
    r = np.asarray(r, dtype=np.float64)
    rho = forgetting_factor(kl, d_half, rho_min, rho_max)
    for j in range(len(ids)):
        i = int(ids[j])
        alpha[i] = rho[j] * alpha[i] + r[j]
        beta[i] = rho[j] * beta[i] + (1.0 - r[j])
    return alpha, beta


def ema_update(v_prev, n_prev, r, rho):
    """EMA restatement of the same update (Sec. 3.1, second display).

    v = v_prev + eta*(r - v_prev) with eta = 1/(rho*n_prev + 1), where n_prev is
    alpha+beta before the update.  (The paper's "N_eff = alpha+beta+1" next to
    this formula does not satisfy the Beta update by algebra; the Beta update is
    taken as the definition and eta is what it implies.)
    """
    eta = 1.0 / (rho * n_prev + 1.0)
    return v_prev + eta * (r - v_prev)


# --------------------------------------------------------------------------
# Sec. 3.2 -- advantage and global normalisation
# --------------------------------------------------------------------------

def raw_advantage(alpha, beta, ids, r):
    """A = r - v_{-1}(x): the table is read before this batch's update (Sec. 3.2)."""
    v = value_estimate(alpha, beta)
    ids = np.asarray(ids, dtype=np.int64)
    return np.asarray(r, dtype=np.float64) - v[ids]


def normalise_advantages(a, ddof=0, eps=1e-8):
    """A~ = (A - mu_B)/sigma_B over the whole batch (Sec. 3.2).

    Population standard deviation by default; ``eps`` is added to sigma so that
    an all-equal batch gives zeros.  Returns (A~, mu, sigma).
    """
    a = np.asarray(a, dtype=np.float64)
    b = a.shape[0]
    if b == 0:
        return a.copy(), 0.0, 0.0
    mu = a.sum() / b
    denom = b - ddof
    if denom <= 0:
        sigma = 0.0
    else:
        sigma = float(np.sqrt(((a - mu) ** 2).sum() / denom))
    return (a - mu) / (sigma + eps), float(mu), sigma


def near_zero_counts(a_raw, taus=(1e-4, 0.02)):
    """How many raw advantages satisfy |A| <= tau, for each tolerance (Sec. 4, "Signal Efficiency
    and Information Loss": the share of near-zero advantages is tracked on the unnormalised
    advantages at tau = 1e-4 and tau = 0.02)."""
    a = np.abs(np.asarray(a_raw, dtype=np.float64))
    return [int((a <= float(t)).sum()) for t in taus]


# --------------------------------------------------------------------------
# Sec. 3.3 -- prioritised sampling
# --------------------------------------------------------------------------

def sampling_weights(alpha, beta, eps_explore=EPS_EXPLORE):
    """w = sqrt(v(1-v)) + eps (Eq. "sampling_coef"), unnormalised."""
    v = value_estimate(alpha, beta)
    return np.sqrt(v * (1.0 - v)) + float(eps_explore)


def quantise_weights(w32):
    """q = floor(w * 2^32) as unsigned 64-bit integers (exact: a power-of-two scale)."""
    w = np.asarray(w32, dtype=np.float32).astype(np.float64)
    if np.any(w < 0) or not np.all(np.isfinite(w)):
        raise ValueError("weights must be finite and non-negative")
    return np.floor(w * 4294967296.0).astype(np.uint64)


def sample_prompts(w32, uniforms32, batch):
    """Draw ``batch`` distinct prompts by weight (Algorithm 1, "Sample a batch ... according to weights").

    Successive weighted sampling without replacement, realised as inverse-CDF
    draws with replacement whose repeats are skipped (equal in distribution to
    removing each chosen prompt and renormalising).  The CDF is over integers:
    q_i = floor(w_i*2^32), C_i = q_0+...+q_i, Wtot = C_{N-1}.  For the k-th
    uniform u_k in [0,1): U_k = floor(u_k*2^32), t_k = floor(U_k*Wtot / 2^32),
    candidate = the first i with C_i > t_k.  Candidates are accepted in order
    unless already accepted; stops at ``batch`` accepted.  Raises if the
    uniforms run out.  Returns int64 ids in acceptance order.
    """
    q = quantise_weights(w32)
    csum = np.cumsum(q, dtype=np.uint64)
    wtot = int(csum[-1]) if len(csum) else 0
    if wtot == 0:
        raise ValueError("total weight is zero")
    u = np.asarray(uniforms32, dtype=np.float32).astype(np.float64)
    if np.any(u < 0.0) or np.any(u >= 1.0):
        raise ValueError("uniforms must lie in [0,1)")
    chosen = []
    seen = set()
    for k in range(len(u)):
        if len(chosen) == batch:
            break
        big_u = int(np.floor(u[k] * 4294967296.0))
        t = (big_u * wtot) >> 32
        i = int(np.searchsorted(csum, np.uint64(t), side="right"))
        if i not in seen:
            seen.add(i)
            chosen.append(i)
    if len(chosen) < batch:
        raise RuntimeError("not enough uniforms to accept %d distinct prompts" % batch)
    return np.asarray(chosen, dtype=np.int64)


# --------------------------------------------------------------------------
# Sec. 3.2 -- PPO-Clip objective on log-probs from the LM head
# --------------------------------------------------------------------------

def token_sequence_ids(cu_seqlens, n_tokens):
    """seq(t) for packed rows: the s with cu_seqlens[s] <= t < cu_seqlens[s+1]."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    t = np.arange(n_tokens, dtype=np.int64)
    return np.searchsorted(cu, t, side="right") - 1


def logits(h, w):
    """z[t, v] = sum_k W[v, k] * H[t, k] (the LM head; no bias, temperature 1)."""
    return np.asarray(h, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T


AGG_TOKEN_MEAN = 0      # mean over all unmasked tokens of the batch
AGG_SEQ_MEAN = 1        # mean over responses of each response's own token mean


def aggregation_weights(mask01, seq, n_seq, agg_mode):
    """Weight u_t of token t in the expectation E_{s,t} of the objective; the weights sum to 1.

    The paper writes E_{s,t} without saying how tokens of responses of different
    length are weighted.  Mode 0 (the reading taken as default): every unmasked token
    counts alike, u_t = m_t / n_tok.  Mode 1: every response that has an unmasked
    token counts alike and its tokens share its weight, u_t = m_t / (S_act * n_s(t)).
    """
    m = np.asarray(mask01, dtype=np.float64)
    if agg_mode == AGG_TOKEN_MEAN:
        n_tok = m.sum()
        return m / n_tok if n_tok > 0 else np.zeros_like(m)
    if agg_mode == AGG_SEQ_MEAN:
        per_seq = np.zeros(n_seq, dtype=np.float64)
        np.add.at(per_seq, seq, m)
        s_act = float((per_seq > 0).sum())
        if s_act == 0:
            return np.zeros_like(m)
        denom = np.where(per_seq[seq] > 0, per_seq[seq], 1.0)
        return m / (s_act * denom)
    raise ValueError("agg_mode")


SUR_PPO_CLIP = 0        # the paper's objective: token-level PPO-Clip
SUR_CISPO = 1           # clipped importance weight, held constant, times log-prob
SUR_GSPO = 2            # PPO-Clip on one sequence-level ratio per response


def loss_forward(h, w, y, logp_old, mask, cu_seqlens, a_norm,
                 clip_lo=CLIP_LO, clip_hi=CLIP_HI, agg_mode=AGG_TOKEN_MEAN, surrogate=SUR_PPO_CLIP,
                 dual_clip=None):
    """Token-level PPO-Clip surrogate of Sec. 3.2 with Clip-Higher bounds.

    Per token t (row of ``h``): z = W h_t; lse = log sum_v exp(z_v);
    logp = z[y_t] - lse; ratio = exp(logp - logp_old_t); a = A~[seq(t)];
    s = min(ratio*a, clip(ratio, 1-clip_lo, 1+clip_hi)*a).
    The expectation over (s,t) is read as the mean over all unmasked tokens of
    the batch, n_tok = sum(mask); the exported loss is the negated objective.

    Sec. 3.2 closes by naming two other objectives the advantage estimator is
    compatible with, without writing them out; ``surrogate`` selects them in
    the form their own publications give (this implementation's reading):
      SUR_CISPO  the importance ratio is truncated to [1-clip_lo, 1+clip_hi] and
                 enters as a constant weight (no gradient through it) on the
                 log-prob: term_t = w_t * a * logp_t, w_t = clip(ratio_t);
                 so d loss / d logp_t = -u_t * w_t * a for every unmasked token.
      SUR_GSPO   one ratio per response, the geometric mean of its unmasked
                 tokens' ratios: r_i = exp(mean_t (logp_t - logp_old_t));
                 term_i = min(r_i*a_i, clip(r_i)*a_i); the objective is the mean
                 of term_i over the responses that have an unmasked token
                 (``agg_mode`` does not apply), and
                 d loss / d logp_t = -(1/S_act) * a_i * r_i * [unclipped_i] / n_i.
                 ``ratio``, ``surrogate`` and ``unclipped`` then hold each
                 token's response-level value.

    ``dual_clip`` = c > 1 adds the second clip of dual-clip PPO (not in the paper; a variant
    of its objective in the published form): for a negative advantage the term becomes
    max(min(ratio*a, clip(ratio)*a), c*a), which stops the gradient once ratio > c (the
    term is then the constant c*a); non-negative advantages are untouched.  It applies to
    SUR_PPO_CLIP (per token) and SUR_GSPO (per response); SUR_CISPO has its own truncation.

    Returns a dict: loss, logp[T], lse[T], ratio[T], surrogate[T], unclipped[T]
    (bool: the gradient passes through the ratio), coef[T] = d loss / d logp_t
    = -u_t*a*ratio*unclipped with u_t the aggregation weight (mask/n_tok by
    default, see aggregation_weights), n_tok, seq_sums[S,3] = per sequence
    (sum mask*logp, sum mask*(logp_old - logp), sum mask), and entropy[T] =
    -sum_v p log p of each row's softmax (a diagnostic).
    """
    z = logits(h, w)
    n_tok_rows = z.shape[0]
    y = np.asarray(y, dtype=np.int64)
    logp_old = np.asarray(logp_old, dtype=np.float64)
    if mask is None:
        m = np.ones(n_tok_rows, dtype=np.float64)
    else:
        m = (np.asarray(mask) != 0).astype(np.float64)
    zmax = z.max(axis=1) if z.shape[1] else np.zeros(n_tok_rows)
    lse = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    logp = z[np.arange(n_tok_rows), y] - lse
    # entropy of the policy's next-token distribution, -sum_v p log p = lse - sum_v p z (a diagnostic;
    # Sec. 3.2 speaks of retaining policy entropy; it does not enter the objective)
    p_full = np.exp(z - lse[:, None])
    entropy = lse - (p_full * z).sum(axis=1)
    ratio = np.exp(logp - logp_old)
    seq = token_sequence_ids(cu_seqlens, n_tok_rows)
    a = np.asarray(a_norm, dtype=np.float64)[seq]
    n_tok = m.sum()
    n_seq = len(cu_seqlens) - 1
    seq_sums = np.zeros((n_seq, 3), dtype=np.float64)
    np.add.at(seq_sums[:, 0], seq, m * logp)
    np.add.at(seq_sums[:, 1], seq, m * (logp_old - logp))
    np.add.at(seq_sums[:, 2], seq, m)
    lo_b, hi_b = 1.0 - clip_lo, 1.0 + clip_hi
    if surrogate == SUR_GSPO:
        n_i = seq_sums[:, 2]
        live = n_i > 0
        s_act = float(live.sum())
        r_i = np.exp(-seq_sums[:, 1] / np.where(live, n_i, 1.0))          # exp(mean(logp - logp_old))
        a_i = np.asarray(a_norm, dtype=np.float64)[:n_seq]
        term_i = np.minimum(r_i * a_i, np.minimum(np.maximum(r_i, lo_b), hi_b) * a_i)
        pass_i = np.where(a_i >= 0.0, r_i <= hi_b, r_i >= lo_b)
        if dual_clip is not None:
            neg = a_i < 0.0
            term_i = np.where(neg, np.maximum(term_i, float(dual_clip) * a_i), term_i)
            pass_i = pass_i & ~(neg & (r_i > float(dual_clip)))
        loss = -(term_i[live].sum() / s_act) if s_act > 0 else 0.0
        ratio = r_i[seq]
        surrogate_t = term_i[seq]
        unclipped = pass_i[seq]
        if s_act > 0:
            coef = -(m * a * ratio * unclipped) / (s_act * np.where(n_i[seq] > 0, n_i[seq], 1.0))
        else:
            coef = np.zeros(n_tok_rows)
    else:
        u = aggregation_weights(m, seq, n_seq, agg_mode)
        clipped_ratio = np.minimum(np.maximum(ratio, lo_b), hi_b)
        if surrogate == SUR_CISPO:
            surrogate_t = clipped_ratio * a * logp
            unclipped = np.ones(n_tok_rows, dtype=bool)
            coef = -(u * clipped_ratio * a)
        elif surrogate == SUR_PPO_CLIP:
            surrogate_t = np.minimum(ratio * a, clipped_ratio * a)
            # The min picks the unclipped branch (and so carries gradient) when the
            # ratio is on the inside of the bound that matters for the sign of a;
            # the boundary itself counts as inside.
            unclipped = np.where(a >= 0.0, ratio <= hi_b, ratio >= lo_b)
            if dual_clip is not None:
                # second clip for negative advantages: the term may not fall below c*a, and once
                # ratio > c it is that constant (ratio == c counts as inside, like the other bounds)
                neg = a < 0.0
                surrogate_t = np.where(neg, np.maximum(surrogate_t, float(dual_clip) * a), surrogate_t)
                unclipped = unclipped & ~(neg & (ratio > float(dual_clip)))
            coef = -(u * a * ratio * unclipped)
        else:
            raise ValueError("surrogate")
        loss = -(u * surrogate_t).sum()
    return {
        "loss": float(loss), "logp": logp, "lse": lse, "ratio": ratio,
        "surrogate": surrogate_t, "unclipped": unclipped, "coef": coef,
        "n_tok": float(n_tok), "seq_sums": seq_sums, "entropy": entropy,
    }


def loss_stats(logp, logp_old, mask, cu_seqlens, a_norm, clip_lo=CLIP_LO, clip_hi=CLIP_HI, dual_clip=None):
    """Per-step diagnostics of the policy update over the unmasked tokens (the quantities the
    paper's training curves are read by; none enters the objective):
      [0] n_tok            [1] mean importance ratio
      [2] share of tokens whose gradient the clip stops (ratio beyond the bound that matters
          for the sign of their advantage, or beyond ``dual_clip`` for a negative one; a zero
          advantage counts as not clipped)
      [3] mean of logp_old - logp            (the plain sampled estimate of KL(old || new))
      [4] mean of ratio - 1 - log(ratio)     (a non-negative estimate of the same KL)
      [5] largest ratio    [6] smallest ratio
      [7] share of tokens whose ratio lies outside [1-clip_lo, 1+clip_hi], whatever the sign.
    All zeros when no token is unmasked.
    """
    logp = np.asarray(logp, dtype=np.float64)
    logp_old = np.asarray(logp_old, dtype=np.float64)
    t = logp.shape[0]
    m = np.ones(t, dtype=bool) if mask is None else (np.asarray(mask) != 0)
    out = np.zeros(8, dtype=np.float64)
    n = int(m.sum())
    if n == 0:
        return out
    seq = token_sequence_ids(cu_seqlens, t)
    a = np.asarray(a_norm, dtype=np.float64)[seq][m]
    d = (logp - logp_old)[m]
    ratio = np.exp(d)
    lo_b, hi_b = 1.0 - clip_lo, 1.0 + clip_hi
    stopped = np.where(a > 0.0, ratio > hi_b, np.where(a < 0.0, ratio < lo_b, False))
    if dual_clip is not None:
        stopped = stopped | ((a < 0.0) & (ratio > float(dual_clip)))
    out[0] = n
    out[1] = ratio.mean()
    out[2] = stopped.mean()
    out[3] = (-d).mean()
    out[4] = (ratio - 1.0 - d).mean()
    out[5] = ratio.max()
    out[6] = ratio.min()
    out[7] = ((ratio > hi_b) | (ratio < lo_b)).mean()
    return out


def loss_backward(h, w, y, lse, coef, grad_loss=1.0):
    """Gradients of the exported loss with respect to H and W.

    With p = exp(z - lse) (the softmax) the logit gradient is
    g[t, v] = grad_loss * coef_t * (1[v = y_t] - p[t, v]);
    dH = g W ; dW = g^T H.
    """
    h = np.asarray(h, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    z = h @ w.T
    p = np.exp(z - np.asarray(lse, dtype=np.float64)[:, None])
    g = -p
    g[np.arange(z.shape[0]), np.asarray(y, dtype=np.int64)] += 1.0
    g *= (float(grad_loss) * np.asarray(coef, dtype=np.float64))[:, None]
    return g @ w, g.T @ h


def loss_rows(h_rows, w, y_rows, logp_old_rows, mask_rows, a_rows, n_tok,
              clip_lo=CLIP_LO, clip_hi=CLIP_HI, grad_loss=1.0, v_chunk=8192, want_dw=False):
    """Row-local outputs for a handful of token rows of a large problem.

    Every per-token output of loss_forward and the dH row of loss_backward
    depends only on that token's hidden state, W and batch-level scalars
    (the advantage of its sequence, n_tok).  This evaluates exactly those
    formulas for the given rows, streaming W in chunks of ``v_chunk`` rows so
    that W never has to exist in float64 at once.  Returns dict(logp, lse,
    ratio, coef, dH); with ``want_dw`` also dW = g^T H of these rows alone: dW of
    the whole batch is the sum of its tokens' terms, so the contributions of a
    partition of the rows add up to loss_backward's dW.
    """
    h = np.asarray(h_rows, dtype=np.float64)
    n, d = h.shape
    v_total = w.shape[0]
    z = np.empty((n, v_total), dtype=np.float64)
    for v0 in range(0, v_total, v_chunk):
        wc = np.asarray(w[v0:v0 + v_chunk], dtype=np.float64)
        z[:, v0:v0 + wc.shape[0]] = h @ wc.T
    zmax = z.max(axis=1)
    lse = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    y = np.asarray(y_rows, dtype=np.int64)
    logp = z[np.arange(n), y] - lse
    ratio = np.exp(logp - np.asarray(logp_old_rows, dtype=np.float64))
    a = np.asarray(a_rows, dtype=np.float64)
    m = (np.asarray(mask_rows) != 0).astype(np.float64)
    unclipped = np.where(a >= 0.0, ratio <= 1.0 + clip_hi, ratio >= 1.0 - clip_lo)
    coef = -(m * a * ratio * unclipped) / float(n_tok)
    g = -np.exp(z - lse[:, None])
    g[np.arange(n), y] += 1.0
    g *= (float(grad_loss) * coef)[:, None]
    dh = np.zeros((n, d), dtype=np.float64)
    for v0 in range(0, v_total, v_chunk):
        wc = np.asarray(w[v0:v0 + v_chunk], dtype=np.float64)
        dh += g[:, v0:v0 + wc.shape[0]] @ wc
    out = {"logp": logp, "lse": lse, "ratio": ratio, "coef": coef, "dH": dh}
    if want_dw:
        out["dW"] = g.T @ h
    return out
