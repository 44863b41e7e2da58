"""Pins for the CPU oracle: closed forms, hand-worked values, brute force, finite
differences, library routines and the constants the paper prints.  No GPU."""

import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import spo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def paper_constants():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


# ------------------------------------------------------------------ tracker

def test_paper_constants_match_oracle_defaults():
    c = paper_constants()
    assert O.RHO_MIN == c["rho_min"] and O.RHO_MAX == c["rho_max"]
    assert O.EPS_EXPLORE == c["eps_explore"]
    assert O.CLIP_LO == c["clip_low"] and O.CLIP_HI == c["clip_high"]
    assert O.N0_SAMPLES == c["n0"]
    import inspect
    taus = inspect.signature(O.near_zero_counts).parameters["taus"].default
    assert tuple(taus) == (c["near_zero_tau_tight"], c["near_zero_tau_loose"])


def test_init_effective_sample_size_is_window_min():
    c = paper_constants()
    v0 = np.array([0.0, 0.125, 0.5, 1.0])
    a, b = O.tracker_init(v0, c["rho_min"])
    np.testing.assert_allclose(a + b, c["window_min"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(O.value_estimate(a, b), v0, atol=1e-15)


@pytest.mark.parametrize("key_rho,key_win", [("rho_min", "window_min"), ("rho_max", "window_max")])
def test_equilibrium_window_sizes(key_rho, key_win):
    """alpha+beta converges to 1/(1-rho): 8 at rho_min and 25 at rho_max."""
    c = paper_constants()
    rho = c[key_rho]
    d_half = 1.0
    kl = -math.log2(rho) * d_half          # 2^(-kl/d_half) == rho, inside the clamp
    a, b = np.array([3.0]), np.array([1.0])
    rng = np.random.default_rng(0)
    for _ in range(600):
        r = float(rng.random() < 0.3)
        a, b = O.tracker_update(a, b, [0], [r], [kl], d_half, c["rho_min"], c["rho_max"])
    assert abs((a + b)[0] - c[key_win]) < 1e-6


def test_equilibrium_start_is_fixed_point_and_constant_reward_closed_form():
    rho, c_reward, v0 = 0.875, 1.0, 0.25
    a, b = O.tracker_init(np.array([v0]), rho)
    kl = -math.log2(rho) * 0.1
    for k in range(1, 40):
        a, b = O.tracker_update(a, b, [0], [c_reward], [kl], 0.1, 0.875, 0.96)
        assert abs((a + b)[0] - 8.0) < 1e-12
        expect = c_reward + rho ** k * (v0 - c_reward)
        assert abs(O.value_estimate(a, b)[0] - expect) < 1e-12
    # the estimate is driven to the constant reward
    for _ in range(400):
        a, b = O.tracker_update(a, b, [0], [c_reward], [kl], 0.1, 0.875, 0.96)
    assert abs(O.value_estimate(a, b)[0] - 1.0) < 1e-9


def test_constant_zero_reward_drives_estimate_to_zero():
    a, b = O.tracker_init(np.array([0.9]), 0.875)
    for _ in range(300):
        a, b = O.tracker_update(a, b, [0], [0.0], [0.05], 0.1)
    assert O.value_estimate(a, b)[0] < 1e-9


def test_rho_one_is_beta_bernoulli_counting():
    """With no forgetting the update is the textbook conjugate count update."""
    rs = [1, 0, 0, 1, 1, 1, 0]
    a, b = np.array([2.0]), np.array([5.0])
    for r in rs:
        a, b = O.tracker_update(a, b, [0], [float(r)], [0.0], 1.0, rho_min=0.0, rho_max=1.0)
    assert a[0] == 2.0 + sum(rs) and b[0] == 5.0 + len(rs) - sum(rs)
    post = scipy.stats.beta(2.0 + sum(rs), 5.0 + len(rs) - sum(rs))
    assert abs(O.value_estimate(a, b)[0] - post.mean()) < 1e-15


def test_forgetting_factor_values_and_clamp():
    # 2^(-1) = 0.5 is below rho_min; 2^0 = 1 above rho_max; 2^(-1/8) is inside.
    rho = O.forgetting_factor([1.0, 0.0, 0.125, -3.0], 1.0, 0.875, 0.96)
    np.testing.assert_allclose(rho, [0.875, 0.96, 0.9170040432046712, 0.96], atol=1e-15)
    # halving: D = D_half halves the memory when the clamp is open
    assert O.forgetting_factor([0.3], 0.3, 0.0, 1.0)[0] == 0.5


def test_bayes_update_equals_ema_form():
    rng = np.random.default_rng(1)
    for _ in range(50):
        a0, b0 = rng.uniform(0.1, 20, 2)
        r = float(rng.random() < 0.5)
        kl = rng.lognormal(-4, 1)
        rho = O.forgetting_factor([kl], 0.1)[0]
        a, b = O.tracker_update([a0], [b0], [0], [r], [kl], 0.1)
        ema = O.ema_update(a0 / (a0 + b0), a0 + b0, r, rho)
        assert abs(O.value_estimate(a, b)[0] - ema) < 1e-14
        # the learning rate is one over the new effective sample size
        assert abs(1.0 / (rho * (a0 + b0) + 1.0) - 1.0 / (a + b)[0]) < 1e-15


def test_update_touches_only_batch_rows_and_keeps_domain():
    rng = np.random.default_rng(2)
    a0, b0 = rng.uniform(0, 5, 10), rng.uniform(0, 5, 10)
    ids = [7, 2, 5]
    a, b = O.tracker_update(a0, b0, ids, [1.0, 0.0, 1.0], [0.01, 0.2, 5.0], 0.1)
    untouched = [i for i in range(10) if i not in ids]
    assert np.array_equal(a[untouched], a0[untouched]) and np.array_equal(b[untouched], b0[untouched])
    assert np.all(a >= 0) and np.all(b >= 0)
    v = O.value_estimate(a, b)
    assert np.all((v >= 0) & (v <= 1))
    # one row by hand: kl=5 -> rho clamps to 0.875; r=1
    assert abs(a[5] - (0.875 * a0[5] + 1.0)) < 1e-15 and abs(b[5] - 0.875 * b0[5]) < 1e-15
    # r=0 row by hand: kl = 0.2, d_half 0.1 -> 2^-2 = 0.25 -> clamp 0.875
    assert abs(a[2] - 0.875 * a0[2]) < 1e-15 and abs(b[2] - (0.875 * b0[2] + 1.0)) < 1e-15


def test_empty_tracker_estimates_half_then_first_reward():
    assert O.value_estimate([0.0], [0.0])[0] == 0.5
    a, b = O.tracker_update([0.0], [0.0], [0], [1.0], [0.01], 0.1)
    assert O.value_estimate(a, b)[0] == 1.0


# ---------------------------------------------------------------- advantage

def test_no_baseline_table_gives_reward_as_advantage():
    a, b = np.zeros(4), np.ones(4)            # v = 0 everywhere
    r = np.array([1.0, 0.0, 1.0, 1.0])
    np.testing.assert_array_equal(O.raw_advantage(a, b, [3, 1, 0, 2], r), r)


def test_advantage_uses_table_rows_by_id():
    a, b = np.array([1.0, 3.0, 1.0]), np.array([3.0, 1.0, 1.0])   # v = .25 .75 .5
    out = O.raw_advantage(a, b, [2, 0, 1], [1.0, 1.0, 0.0])
    np.testing.assert_allclose(out, [0.5, 0.75, -0.75], atol=1e-15)


@pytest.mark.parametrize("ddof", [0, 1])
def test_normalisation_against_library_zscore(ddof):
    rng = np.random.default_rng(3)
    a = rng.uniform(-1, 1, 257)
    out, mu, sigma = O.normalise_advantages(a, ddof=ddof, eps=0.0)
    np.testing.assert_allclose(out, scipy.stats.zscore(a, ddof=ddof), atol=1e-12)
    assert abs(out.mean()) < 1e-12
    assert abs(out.std(ddof=ddof) - 1.0) < 1e-12
    assert abs(mu - a.mean()) < 1e-15 and abs(sigma - a.std(ddof=ddof)) < 1e-15


def test_normalisation_affine_invariance_and_degenerate_cases():
    rng = np.random.default_rng(4)
    a = rng.uniform(-1, 1, 64)
    base, _, _ = O.normalise_advantages(a, eps=0.0)
    moved, _, _ = O.normalise_advantages(3.5 * a - 2.0, eps=0.0)
    np.testing.assert_allclose(moved, base, atol=1e-12)
    flat, _, sigma = O.normalise_advantages(np.full(9, 0.3))
    assert sigma == 0.0 and np.all(flat == 0.0)
    one, _, _ = O.normalise_advantages(np.array([0.7]))
    assert one[0] == 0.0


# ----------------------------------------------------------------- sampling

def test_near_zero_counts_hand_values_and_tolerances_of_the_paper():
    """Sec. 4 tracks |A| <= tau on the raw advantages at tau = 1e-4 and 0.02; the bound is inclusive."""
    a = np.array([0.0, 1e-4, -1e-4, 1.0001e-4, 0.02, -0.020001, 0.5, -0.7])
    assert O.near_zero_counts(a) == [3, 5]
    assert O.near_zero_counts(a, taus=(0.0, 1.0)) == [1, 8]
    assert O.near_zero_counts([]) == [0, 0]
    # a tracker that predicts perfectly leaves every advantage at zero
    al, be = np.array([8.0, 0.0]), np.array([0.0, 8.0])
    assert O.near_zero_counts(O.raw_advantage(al, be, [0, 1], [1.0, 0.0])) == [2, 2]


def test_weight_range_endpoints():
    eps = paper_constants()["eps_explore"]
    a = np.array([0.0, 8.0, 4.0])
    b = np.array([8.0, 0.0, 4.0])
    w = O.sampling_weights(a, b, eps)
    np.testing.assert_allclose(w, [eps, eps, 0.5 + eps], atol=1e-15)
    rng = np.random.default_rng(5)
    aa, bb = rng.uniform(0, 10, 1000), rng.uniform(0, 10, 1000)
    ww = O.sampling_weights(aa, bb, eps)
    assert ww.min() >= eps and ww.max() <= 0.5 + eps + 1e-15


def test_quantised_weights_are_exact_scalings():
    w = np.array([0.05, 0.55, 0.3, 2.0 ** -8], dtype=np.float32)
    q = O.quantise_weights(w)
    for wi, qi in zip(w, q):
        assert int(qi) == int(Fraction(float(wi)) * 2 ** 32)     # exact rational floor


def _first_index_by_rationals(w32, u):
    q = [int(Fraction(float(x)) * 2 ** 32) for x in w32]
    tot = sum(q)
    c = 0
    for i, qi in enumerate(q):
        c += qi
        if Fraction(c, tot) > Fraction(float(u)):
            return i
    raise AssertionError


def test_first_draw_matches_exact_rational_inverse_cdf():
    rng = np.random.default_rng(7)
    for n in (1, 2, 3, 6):
        w = rng.uniform(0.05, 0.55, n).astype(np.float32)
        if n >= 3:
            w[1] = 0.0                      # a zero weight can never be chosen
        us = np.concatenate([rng.random(300), [0.0, 1 - 2.0 ** -24]]).astype(np.float32)
        us = us[us < 1.0]
        for u in us:
            got = O.sample_prompts(w, [u], 1)[0]
            assert got == _first_index_by_rationals(w, u)
            assert w[got] > 0


def test_equal_weights_systematic_uniforms_hit_every_index():
    n = 64
    w = np.full(n, 0.25, dtype=np.float32)
    u = ((np.arange(n) + 0.5) / n).astype(np.float32)
    np.testing.assert_array_equal(O.sample_prompts(w, u, n), np.arange(n))


def test_repeats_are_skipped_and_full_batch_is_a_permutation():
    w = np.array([0.5, 0.25, 0.25], dtype=np.float32)
    u = np.array([0.1, 0.2, 0.6, 0.55, 0.9], dtype=np.float32)
    np.testing.assert_array_equal(O.sample_prompts(w, u, 3), [0, 1, 2])
    rng = np.random.default_rng(8)
    ww = rng.uniform(0.05, 0.55, 40).astype(np.float32)
    ids = O.sample_prompts(ww, rng.random(4000).astype(np.float32), 40)
    assert sorted(ids.tolist()) == list(range(40))
    with pytest.raises(RuntimeError):
        O.sample_prompts(w, np.array([0.1, 0.2], dtype=np.float32), 3)


def test_first_draw_frequencies_chi_square():
    rng = np.random.default_rng(9)
    n, draws = 64, 100_000
    a = rng.uniform(0, 8, n).astype(np.float32)
    b = rng.uniform(0, 8, n).astype(np.float32)
    w = O.sampling_weights(a, b).astype(np.float32)         # the selector takes fp32 weights as an input
    u = rng.random(draws).astype(np.float32)
    u = u[u < 1.0]
    counts = np.zeros(n)
    for x in u:
        counts[O.sample_prompts(w, [x], 1)[0]] += 1
    p = w.astype(np.float64) / w.astype(np.float64).sum()
    chi2 = ((counts - len(u) * p) ** 2 / (len(u) * p)).sum()
    assert chi2 < scipy.stats.chi2.ppf(0.9999, n - 1)


def test_successive_sampling_pair_frequencies():
    """Ordered pairs (i,j) appear with probability p_i * p_j / (1 - p_i)."""
    rng = np.random.default_rng(10)
    w = np.array([0.55, 0.05, 0.3, 0.2, 0.4], dtype=np.float32)
    p = w.astype(np.float64) / w.astype(np.float64).sum()
    draws = 40_000
    counts = np.zeros((5, 5))
    for _ in range(draws):
        u = rng.random(64).astype(np.float32)
        u = u[u < 1.0]
        i, j = O.sample_prompts(w, u, 2)
        counts[i, j] += 1
    expect = draws * np.outer(p, p) / (1 - p)[:, None]
    off = ~np.eye(5, dtype=bool)
    assert counts[~off].sum() == 0
    chi2 = ((counts[off] - expect[off]) ** 2 / expect[off]).sum()
    assert chi2 < scipy.stats.chi2.ppf(0.9999, 19)


# --------------------------------------------------------------------- loss

def _identity_problem(z, y, logp_old, a_tok):
    """H = I makes the logits equal to W^T, so arbitrary logits can be fed in."""
    t, v = z.shape
    h = np.eye(t)
    w = z.T.copy()
    cu = np.arange(t + 1)          # one token per sequence -> per-token advantage
    return h, w, np.asarray(y), np.asarray(logp_old), None, cu, np.asarray(a_tok)


def test_uniform_logits_give_minus_log_v():
    t, d, v = 5, 7, 33
    h = np.random.default_rng(11).standard_normal((t, d))
    out = O.loss_forward(h, np.zeros((v, d)), [0, 5, 32, 7, 1], np.zeros(t), None, [0, 2, 5], [1.0, -1.0])
    np.testing.assert_allclose(out["logp"], -math.log(v), atol=1e-14)
    np.testing.assert_allclose(out["lse"], math.log(v), atol=1e-14)


def test_logp_against_naive_softmax_and_library_and_shift_invariance():
    rng = np.random.default_rng(12)
    z = rng.standard_normal((6, 9)) * 3
    y = rng.integers(0, 9, 6)
    args = _identity_problem(z, y, np.zeros(6), np.ones(6))
    out = O.loss_forward(*args)
    naive = np.log(np.exp(z[np.arange(6), y]) / np.exp(z).sum(axis=1))
    np.testing.assert_allclose(out["logp"], naive, atol=1e-13)
    np.testing.assert_allclose(out["lse"], scipy.special.logsumexp(z, axis=1), atol=1e-13)
    shifted = O.loss_forward(*_identity_problem(z + 1000.0, y, np.zeros(6), np.ones(6)))
    np.testing.assert_allclose(shifted["logp"], out["logp"], atol=1e-10)
    # one dominant logit -> probability one
    z2 = np.zeros((1, 9)); z2[0, 4] = 80.0
    assert abs(O.loss_forward(*_identity_problem(z2, [4], [0.0], [1.0]))["logp"][0]) < 1e-30


def test_logits_orientation_is_w_times_h():
    """z[t,v] = <W[v,:], H[t,:]> -- a transposed operand would fail this."""
    h = np.array([[1.0, 2.0]])
    w = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    np.testing.assert_array_equal(O.logits(h, w), [[1.0, 2.0, 3.0]])


def test_ratio_one_gives_minus_mean_advantage():
    rng = np.random.default_rng(13)
    t, d, v = 12, 5, 17
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d))
    y = rng.integers(0, v, t)
    cu = [0, 3, 4, 12]
    a = np.array([0.7, -1.3, 0.2])
    mask = np.array([1, 1, 0, 1, 1, 1, 1, 0, 1, 1, 1, 1], dtype=np.uint8)
    first = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)
    out = O.loss_forward(h, w, y, first["logp"], mask, cu, a)
    np.testing.assert_allclose(out["ratio"], 1.0, atol=1e-15)
    a_tok = np.repeat(a, np.diff(cu))
    assert abs(out["loss"] + (mask * a_tok).sum() / mask.sum()) < 1e-14
    assert out["n_tok"] == 10
    np.testing.assert_allclose(out["seq_sums"][:, 2], [2, 1, 7])
    np.testing.assert_allclose(out["seq_sums"][:, 1], 0.0, atol=1e-13)
    np.testing.assert_allclose(out["seq_sums"][:, 0],
                               [(mask * out["logp"])[lo:hi].sum() for lo, hi in zip(cu[:-1], cu[1:])], atol=1e-13)


def test_clip_branches_hand_worked():
    """Clip-Higher bounds 0.8 / 1.28; hand-computed surrogate and gradient gate."""
    cases = [  # ratio, advantage, surrogate, gradient passes
        (1.5, 1.0, 1.28, False),
        (1.5, -1.0, -1.5, True),
        (0.5, 1.0, 0.5, True),
        (0.5, -1.0, -0.8, False),
        (1.0, 2.0, 2.0, True),
        (1.28, 1.0, 1.28, True),     # boundary counts as inside
        (0.8, -1.0, -0.8, True),
        (1.1, 0.0, 0.0, True),
    ]
    for ratio, adv, s_expect, passes in cases:
        z = np.zeros((1, 4))
        logp_new = -math.log(4)
        logp_old = logp_new - math.log(ratio)
        out = O.loss_forward(*_identity_problem(z, [2], [logp_old], [adv]))
        assert abs(out["ratio"][0] - ratio) < 1e-12
        assert abs(out["surrogate"][0] - s_expect) < 1e-12, (ratio, adv)
        assert abs(out["loss"] + s_expect) < 1e-12
        if ratio not in (1.28, 0.8):       # exactly on the boundary rounding may fall either side
            assert bool(out["unclipped"][0]) == passes
        expect_coef = -adv * ratio if passes else 0.0
        if ratio not in (1.28, 0.8):
            assert abs(out["coef"][0] - expect_coef) < 1e-12


def test_logit_gradient_is_advantage_times_softmax_minus_onehot():
    rng = np.random.default_rng(14)
    t, v = 5, 8
    z = rng.standard_normal((t, v))
    y = rng.integers(0, v, t)
    a = np.array([1.0, -0.5, 2.0, 0.3, -1.2])
    probe = O.loss_forward(*_identity_problem(z, y, np.zeros(t), a))
    # tokens 0..2 at ratio 1 (inside), token 3 clipped from above (a>0), token 4 clipped from below (a<0)
    logp_old = probe["logp"].copy()
    logp_old[3] -= math.log(1.6)
    logp_old[4] += math.log(2.0)
    args = _identity_problem(z, y, logp_old, a)
    fwd = O.loss_forward(*args)
    _, dw = O.loss_backward(args[0], args[1], y, fwd["lse"], fwd["coef"])
    g = dw.T                                   # H = I  ->  dW = g^T
    p = scipy.special.softmax(z, axis=1)
    onehot = np.eye(v)[y]
    expect = a[:, None] * (p - onehot) / t
    np.testing.assert_allclose(g[:3], expect[:3], atol=1e-14)
    assert np.all(g[3:] == 0.0)
    np.testing.assert_allclose(g.sum(axis=1), 0.0, atol=1e-15)


def test_gradients_against_central_finite_differences():
    rng = np.random.default_rng(15)
    t, d, v = 7, 6, 11
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d)) * 0.5
    y = rng.integers(0, v, t)
    cu = [0, 2, 7]
    a = np.array([0.9, -1.1])
    mask = np.array([1, 1, 1, 0, 1, 1, 1], dtype=np.uint8)
    base = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)
    # offsets chosen so that tokens 1 (a>0, ratio 1.5) and 5 (a<0, ratio 0.6) clip; none sits on a bound
    logp_old = base["logp"] - np.log([1.1, 1.5, 0.7, 1.0, 1.2, 0.6, 0.9])
    fwd = O.loss_forward(h, w, y, logp_old, mask, cu, a)
    assert 0 < fwd["unclipped"].sum() < t
    gl = 1.7
    dh, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"], grad_loss=gl)

    def loss_at(hh, ww):
        return gl * O.loss_forward(hh, ww, y, logp_old, mask, cu, a)["loss"]

    step = 1e-6
    for arr, grad in ((h, dh), (w, dw)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + step
            up = loss_at(h, w)
            arr[idx] = keep - step
            dn = loss_at(h, w)
            arr[idx] = keep
            num[idx] = (up - dn) / (2 * step)
        assert np.linalg.norm(num - grad) <= 1e-6 * np.linalg.norm(grad)
    assert np.all(dh[3] == 0.0)                              # masked token


def test_backward_matches_library_autograd():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(16)
    t, d, v = 9, 4, 13
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d))
    y = rng.integers(0, v, t)
    cu, a = [0, 4, 9], np.array([1.0, -0.6])
    logp_old = O.loss_forward(h, w, y, np.zeros(t), None, cu, a)["logp"] + rng.normal(0, 0.2, t)
    fwd = O.loss_forward(h, w, y, logp_old, None, cu, a)
    dh, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"])
    ht = torch.tensor(h, requires_grad=True)
    wt = torch.tensor(w, requires_grad=True)
    lp = torch.log_softmax(ht @ wt.T, dim=1)[torch.arange(t), torch.tensor(y)]
    ratio = torch.exp(lp - torch.tensor(logp_old))
    at = torch.tensor(np.repeat(a, np.diff(cu)))
    loss = -torch.minimum(ratio * at, torch.clamp(ratio, 0.8, 1.28) * at).mean()
    loss.backward()
    assert abs(loss.item() - fwd["loss"]) < 1e-13
    np.testing.assert_allclose(dh, ht.grad.numpy(), atol=1e-13)
    np.testing.assert_allclose(dw, wt.grad.numpy(), atol=1e-13)


def test_row_local_helper_equals_full_definition():
    rng = np.random.default_rng(17)
    t, d, v = 20, 8, 50
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d))
    y = rng.integers(0, v, t)
    cu, a = [0, 5, 20], np.array([0.4, -1.5])
    mask = (rng.random(t) > 0.2).astype(np.uint8)
    logp_old = rng.normal(-4, 0.3, t)
    fwd = O.loss_forward(h, w, y, logp_old, mask, cu, a)
    dh, _ = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"], grad_loss=0.5)
    rows = [0, 4, 5, 19]
    a_tok = np.repeat(a, np.diff(cu))
    sub = O.loss_rows(h[rows], w, y[rows], logp_old[rows], mask[rows], a_tok[rows], fwd["n_tok"],
                      grad_loss=0.5, v_chunk=16)
    np.testing.assert_allclose(sub["logp"], fwd["logp"][rows], atol=1e-13)
    np.testing.assert_allclose(sub["lse"], fwd["lse"][rows], atol=1e-13)
    np.testing.assert_allclose(sub["coef"], fwd["coef"][rows], atol=1e-15)
    np.testing.assert_allclose(sub["dH"], dh[rows], atol=1e-14)
    assert "dW" not in sub


def test_row_local_dw_contributions_of_a_partition_add_up_to_the_full_dw():
    """dW = g^T H is a sum over tokens: the row blocks' contributions must add up to
    loss_backward's dW (what the multi-chunk parity test at the real vocabulary relies on)."""
    rng = np.random.default_rng(18)
    t, d, v = 23, 6, 40
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d))
    y = rng.integers(0, v, t)
    cu, a = [0, 9, 23], np.array([0.8, -1.3])
    mask = (rng.random(t) > 0.2).astype(np.uint8)
    logp_old = rng.normal(-3.5, 0.3, t)
    fwd = O.loss_forward(h, w, y, logp_old, mask, cu, a)
    _, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"], grad_loss=0.7)
    a_tok = np.repeat(a, np.diff(cu))
    acc = np.zeros_like(dw)
    for lo, hi in ((0, 7), (7, 8), (8, 23)):
        sub = O.loss_rows(h[lo:hi], w, y[lo:hi], logp_old[lo:hi], mask[lo:hi], a_tok[lo:hi], fwd["n_tok"],
                          grad_loss=0.7, v_chunk=16, want_dw=True)
        acc += sub["dW"]
    np.testing.assert_allclose(acc, dw, atol=1e-13)
    # a transposed operand or a dropped block would not survive this: dW is [V, d], not symmetric
    assert acc.shape == (v, d)


def test_token_to_sequence_map():
    np.testing.assert_array_equal(O.token_sequence_ids([0, 2, 2, 5], 5), [0, 0, 2, 2, 2])


# ------------------------------------------------------ aggregation variants

def test_aggregation_weights_sum_to_one_and_hand_values():
    seq = np.array([0, 1, 1, 1, 2, 2])
    m = np.array([1, 1, 0, 1, 0, 0], dtype=float)          # response 2 fully masked
    u0 = O.aggregation_weights(m, seq, 3, O.AGG_TOKEN_MEAN)
    u1 = O.aggregation_weights(m, seq, 3, O.AGG_SEQ_MEAN)
    np.testing.assert_allclose(u0, [1 / 3, 1 / 3, 0, 1 / 3, 0, 0])
    np.testing.assert_allclose(u1, [1 / 2, 1 / 4, 0, 1 / 4, 0, 0])
    assert abs(u0.sum() - 1) < 1e-15 and abs(u1.sum() - 1) < 1e-15
    assert O.aggregation_weights(np.zeros(4), np.zeros(4, int), 1, O.AGG_SEQ_MEAN).sum() == 0.0


def test_sequence_mean_at_ratio_one_is_minus_mean_of_response_advantages():
    rng = np.random.default_rng(21)
    t, d, v = 9, 4, 12
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d))
    y = rng.integers(0, v, t)
    cu, a = [0, 1, 4, 9], np.array([2.0, -1.0, 0.5])
    new = O.loss_forward(h, w, y, np.zeros(t), None, cu, a)["logp"]
    tok = O.loss_forward(h, w, y, new, None, cu, a, agg_mode=O.AGG_TOKEN_MEAN)
    seq = O.loss_forward(h, w, y, new, None, cu, a, agg_mode=O.AGG_SEQ_MEAN)
    assert abs(seq["loss"] + a.mean()) < 1e-14                       # each response counts once
    assert abs(tok["loss"] + (1 * 2.0 - 3 * 1.0 + 5 * 0.5) / 9) < 1e-14  # each token counts once
    # equal lengths: the two readings coincide
    same = [O.loss_forward(h[:8], w, y[:8], new[:8], None, [0, 4, 8], a[:2], agg_mode=k)["loss"] for k in (0, 1)]
    assert abs(same[0] - same[1]) < 1e-15


def test_sequence_mean_gradients_against_finite_differences():
    rng = np.random.default_rng(22)
    t, d, v = 7, 5, 9
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d)) * 0.5
    y = rng.integers(0, v, t)
    cu, a = [0, 2, 3, 7], np.array([0.9, -1.1, 0.4])
    mask = np.array([1, 1, 1, 0, 1, 1, 1], dtype=np.uint8)
    base = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)["logp"]
    logp_old = base - np.log([1.1, 1.5, 0.6, 1.0, 1.2, 0.9, 1.05])
    fwd = O.loss_forward(h, w, y, logp_old, mask, cu, a, agg_mode=O.AGG_SEQ_MEAN)
    dh, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"])
    step = 1e-6
    for arr, grad in ((h, dh), (w, dw)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + step
            up = O.loss_forward(h, w, y, logp_old, mask, cu, a, agg_mode=O.AGG_SEQ_MEAN)["loss"]
            arr[idx] = keep - step
            dn = O.loss_forward(h, w, y, logp_old, mask, cu, a, agg_mode=O.AGG_SEQ_MEAN)["loss"]
            arr[idx] = keep
            num[idx] = (up - dn) / (2 * step)
        assert np.linalg.norm(num - grad) <= 1e-6 * np.linalg.norm(grad)


def test_general_rewards_follow_the_ema_form():
    """Sec. 3.1, last sentence: for non-binary rewards the same EMA tracks the value.  With
    (alpha, beta) carried as before, alpha/(alpha+beta) obeys that EMA for any real reward."""
    rng = np.random.default_rng(23)
    v, n = 0.3, 8.0
    a, b = np.array([v * n]), np.array([(1 - v) * n])
    for _ in range(200):
        r = float(rng.uniform(0.0, 1.0))
        kl = float(rng.lognormal(-4, 1))
        rho = O.forgetting_factor([kl], 0.1)[0]
        v = O.ema_update(v, n, r, rho)
        n = rho * n + 1.0
        a, b = O.tracker_update(a, b, [0], [r], [kl], 0.1)
        assert abs(O.value_estimate(a, b)[0] - v) < 1e-12
        assert abs((a + b)[0] - n) < 1e-12
    # a constant fractional reward is tracked to that reward
    a, b = O.tracker_init(np.array([0.9]), 0.875)
    for _ in range(400):
        a, b = O.tracker_update(a, b, [0], [0.37], [0.05], 0.1)
    assert abs(O.value_estimate(a, b)[0] - 0.37) < 1e-9


def test_repeated_ids_apply_in_batch_order():
    """Batch SPO: several outcomes of one prompt in a batch compose the update in order."""
    a0, b0 = np.array([2.0, 1.0]), np.array([3.0, 4.0])
    ids, r, kl = [0, 1, 0, 0], [1.0, 0.0, 0.0, 1.0], [0.01, 0.02, 0.2, 0.005]
    a, b = O.tracker_update(a0, b0, ids, r, kl, 0.1)
    sa, sb = a0.copy(), b0.copy()
    for j in range(4):                               # one call per entry
        sa, sb = O.tracker_update(sa, sb, [ids[j]], [r[j]], [kl[j]], 0.1)
    np.testing.assert_array_equal(a, sa)
    np.testing.assert_array_equal(b, sb)
    # order matters: swapping the two zero/one rewards of prompt 0 changes the estimate
    a2, b2 = O.tracker_update(a0, b0, [0, 1, 0, 0], [1.0, 0.0, 1.0, 0.0], kl, 0.1)
    assert abs(O.value_estimate(a, b)[0] - O.value_estimate(a2, b2)[0]) > 1e-3
    # every copy of a prompt sees the same pre-update baseline
    adv = O.raw_advantage(a0, b0, ids, r)
    assert adv[0] == 1.0 - 0.4 and adv[2] == 0.0 - 0.4 and adv[3] == 1.0 - 0.4


# ------------------------------------------------------------------ the other objectives Sec. 3.2 names

def _tiny_loss_case(seed, cu, t, d=5, v=9):
    rng = np.random.default_rng(seed)
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d)) * 0.5
    y = rng.integers(0, v, t)
    return h, w, y


def test_cispo_hand_values_and_agreement_with_ppo_clip_inside_the_bounds():
    """Truncated importance weight held constant: coef = -u * clip(ratio) * a for every unmasked token.
    Inside the clip bounds that is PPO-Clip's own gradient; outside, PPO-Clip gives zero on the
    clipped side while this objective keeps the truncated weight."""
    t, cu, a = 6, [0, 3, 6], np.array([2.0, -1.0])
    h, w, y = _tiny_loss_case(31, cu, t)
    mask = np.array([1, 1, 1, 1, 0, 1], dtype=np.uint8)
    base = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)["logp"]
    ratios = np.array([1.0, 1.5, 0.5, 1.1, 1.0, 0.6])
    logp_old = base - np.log(ratios)
    cis = O.loss_forward(h, w, y, logp_old, mask, cu, a, surrogate=O.SUR_CISPO)
    ppo = O.loss_forward(h, w, y, logp_old, mask, cu, a)
    np.testing.assert_allclose(cis["ratio"], ratios, rtol=1e-12)
    # n_tok = 5; weights: 1, 1.28 (cut from 1.5), 0.8 (raised from 0.5), 1.1, -, 0.8 (raised from 0.6)
    want = -np.array([1.0 * 2, 1.28 * 2, 0.8 * 2, 1.1 * -1, 0.0, 0.8 * -1]) / 5.0
    np.testing.assert_allclose(cis["coef"], want, rtol=1e-12, atol=1e-15)
    inside = (ratios >= 0.8) & (ratios <= 1.28)
    np.testing.assert_allclose(cis["coef"][inside], ppo["coef"][inside], rtol=1e-12, atol=1e-15)
    # token 1: a > 0 above the upper bound -> PPO-Clip stops the gradient, the truncated weight does not
    assert ppo["coef"][1] == 0.0 and cis["coef"][1] != 0.0
    # loss = -(1/n_tok) sum w a logp
    wts = np.clip(ratios, 0.8, 1.28)
    a_tok = np.repeat(a, 3)
    assert abs(cis["loss"] + (mask * wts * a_tok * cis["logp"]).sum() / 5.0) < 1e-14


def test_cispo_gradients_are_those_of_the_weighted_log_likelihood():
    """With the weights frozen at their current values the objective is a weighted log-likelihood;
    its central finite differences give dH and dW."""
    t, cu, a = 7, [0, 2, 7], np.array([0.9, -1.1])
    h, w, y = _tiny_loss_case(32, cu, t, d=6, v=11)
    mask = np.array([1, 1, 1, 0, 1, 1, 1], dtype=np.uint8)
    base = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)["logp"]
    logp_old = base - np.log([1.1, 1.5, 0.7, 1.0, 1.2, 0.6, 0.9])
    fwd = O.loss_forward(h, w, y, logp_old, mask, cu, a, surrogate=O.SUR_CISPO)
    dh, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"], grad_loss=1.3)
    frozen = np.clip(fwd["ratio"], 0.8, 1.28) * np.repeat(a, np.diff(cu)) * mask / mask.sum()

    def frozen_loss(hh, ww):
        lp = scipy.special.log_softmax(hh @ ww.T, axis=1)[np.arange(t), y]
        return -1.3 * (frozen * lp).sum()

    step = 1e-6
    for arr, grad in ((h, dh), (w, dw)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + step
            up = frozen_loss(h, w)
            arr[idx] = keep - step
            dn = frozen_loss(h, w)
            arr[idx] = keep
            num[idx] = (up - dn) / (2 * step)
        assert np.linalg.norm(num - grad) <= 1e-6 * np.linalg.norm(grad)


def test_gspo_reduces_to_ppo_clip_for_one_token_responses_and_hand_values():
    """Responses of one token: the sequence-level ratio is the token's ratio, so the objective is the
    sequence-mean PPO-Clip objective.  A response whose tokens all moved by the same log-ratio has
    exactly that ratio."""
    t = 5
    cu, a = [0, 1, 2, 3, 4, 5], np.array([1.0, -0.5, 2.0, -1.5, 0.3])
    h, w, y = _tiny_loss_case(33, cu, t)
    base = O.loss_forward(h, w, y, np.zeros(t), None, cu, a)["logp"]
    logp_old = base - np.log([1.0, 1.5, 0.5, 0.7, 1.4])
    g = O.loss_forward(h, w, y, logp_old, None, cu, a, surrogate=O.SUR_GSPO)
    p = O.loss_forward(h, w, y, logp_old, None, cu, a, agg_mode=O.AGG_SEQ_MEAN)
    assert abs(g["loss"] - p["loss"]) < 1e-14
    np.testing.assert_allclose(g["coef"], p["coef"], rtol=1e-12, atol=1e-16)
    # one response of four tokens, every token's ratio e^0.1; a second, masked out entirely, drops out
    t = 6
    cu, a = [0, 4, 6], np.array([-2.0, 7.0])
    h, w, y = _tiny_loss_case(34, cu, t)
    mask = np.array([1, 1, 0, 1, 0, 0], dtype=np.uint8)
    base = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)["logp"]
    g = O.loss_forward(h, w, y, base - 0.1, mask, cu, a, surrogate=O.SUR_GSPO)
    r = math.exp(0.1)
    np.testing.assert_allclose(g["ratio"][:4], r, rtol=1e-12)
    assert abs(g["loss"] - 2.0 * r) < 1e-12                     # -(min(r*-2, clip(r)*-2)) / 1 response
    np.testing.assert_allclose(g["coef"], np.array([1, 1, 0, 1, 0, 0]) * 2.0 * r / 3.0, rtol=1e-12)
    # geometric mean: ratios 2 and 1/2 on a two-token response give a sequence ratio of 1
    cu, a = [0, 2], np.array([1.0])
    h, w, y = _tiny_loss_case(35, cu, 2)
    base = O.loss_forward(h, w, y, np.zeros(2), None, cu, a)["logp"]
    g = O.loss_forward(h, w, y, base - np.log([2.0, 0.5]), None, cu, a, surrogate=O.SUR_GSPO)
    np.testing.assert_allclose(g["ratio"], 1.0, rtol=1e-12)
    assert abs(g["loss"] + 1.0) < 1e-12


def test_gspo_gradients_against_central_finite_differences():
    t, cu, a = 9, [0, 2, 2, 6, 9], np.array([0.9, 5.0, -1.1, 0.4])
    h, w, y = _tiny_loss_case(36, cu, t, d=6, v=11)
    mask = np.array([1, 1, 1, 0, 1, 1, 1, 1, 1], dtype=np.uint8)
    base = O.loss_forward(h, w, y, np.zeros(t), mask, cu, a)["logp"]
    # response 0: mean log-ratio above the upper bound with a > 0 (clipped); response 2: inside; 3: inside
    logp_old = base - np.log([1.5, 1.4, 0.9, 1.0, 0.95, 0.85, 1.1, 1.2, 0.9])
    fwd = O.loss_forward(h, w, y, logp_old, mask, cu, a, surrogate=O.SUR_GSPO)
    per_seq_pass = [fwd["unclipped"][0], fwd["unclipped"][2], fwd["unclipped"][6]]
    assert per_seq_pass == [False, True, True]
    dh, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"], grad_loss=0.8)
    assert np.all(dh[:2] == 0.0) and np.all(dh[3] == 0.0)

    def loss_at(hh, ww):
        return 0.8 * O.loss_forward(hh, ww, y, logp_old, mask, cu, a, surrogate=O.SUR_GSPO)["loss"]

    step = 1e-6
    for arr, grad in ((h, dh), (w, dw)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + step
            up = loss_at(h, w)
            arr[idx] = keep - step
            dn = loss_at(h, w)
            arr[idx] = keep
            num[idx] = (up - dn) / (2 * step)
        assert np.linalg.norm(num - grad) <= 1e-6 * np.linalg.norm(grad)


def test_loss_stats_hand_values_and_consistency_with_the_objective():
    logp_old = np.log(np.array([0.5, 0.5, 0.5, 0.5, 0.5, 0.5]))
    ratios = np.array([1.0, 1.5, 0.5, 1.1, 7.0, 0.6])
    logp = logp_old + np.log(ratios)
    mask = np.array([1, 1, 1, 1, 0, 1], dtype=np.uint8)
    cu, a = [0, 3, 6], np.array([2.0, -1.0])
    st = O.loss_stats(logp, logp_old, mask, cu, a)
    live = ratios[[0, 1, 2, 3, 5]]
    assert st[0] == 5
    assert abs(st[1] - live.mean()) < 1e-14
    # a > 0: 1.5 is above 1.28 (stopped), 0.5 is below 0.8 but on the side that still carries gradient;
    # a < 0: 1.1 inside, 0.6 below 0.8 (stopped)
    assert abs(st[2] - 2 / 5) < 1e-15
    assert abs(st[3] + np.log(live).mean()) < 1e-14
    assert abs(st[4] - (live - 1 - np.log(live)).mean()) < 1e-14 and st[4] >= 0
    assert st[5] == 1.5 and st[6] == 0.5
    assert abs(st[7] - 3 / 5) < 1e-15
    # the tokens it counts as stopped are the unmasked ones whose coef the objective sets to zero
    h, w, y = _tiny_loss_case(41, cu, 6)
    base = O.loss_forward(h, w, y, np.zeros(6), mask, cu, a)["logp"]
    fwd = O.loss_forward(h, w, y, base - np.log(ratios), mask, cu, a)
    st2 = O.loss_stats(fwd["logp"], base - np.log(ratios), mask, cu, a)
    assert abs(st2[2] - ((fwd["coef"] == 0) & (mask != 0)).sum() / 5) < 1e-15
    # identical policies: ratio 1, both KL estimates 0, nothing clipped; nothing unmasked: zeros
    same = O.loss_stats(logp_old, logp_old, None, cu, a)
    np.testing.assert_allclose(same, [6, 1, 0, 0, 0, 1, 1, 0], atol=1e-15)
    assert np.all(O.loss_stats(logp, logp_old, np.zeros(6, np.uint8), cu, a) == 0)


def test_policy_entropy_against_library_and_closed_forms():
    rng = np.random.default_rng(51)
    t, d, v = 6, 5, 17
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d)) * 2.0
    y = rng.integers(0, v, t)
    cu, a = [0, 6], np.array([1.0])
    fwd = O.loss_forward(h, w, y, np.zeros(t), None, cu, a)
    p = scipy.special.softmax(h @ w.T, axis=1)
    np.testing.assert_allclose(fwd["entropy"], scipy.stats.entropy(p, axis=1), rtol=1e-12)
    # uniform logits: log V; one dominant logit: close to zero; two equal dominant logits: log 2
    flat = O.loss_forward(h, np.zeros((v, d)), y, np.zeros(t), None, cu, a)
    np.testing.assert_allclose(flat["entropy"], math.log(v), rtol=1e-13)
    hh = np.zeros((1, 2)); hh[0, 0] = 1.0
    ww = np.zeros((4, 2)); ww[0, 0] = 60.0; ww[1, 0] = 60.0
    two = O.loss_forward(hh, ww, [0], np.zeros(1), None, [0, 1], a)
    assert abs(two["entropy"][0] - math.log(2.0)) < 1e-12
    ww[1, 0] = 0.0
    one = O.loss_forward(hh, ww, [0], np.zeros(1), None, [0, 1], a)
    assert 0.0 <= one["entropy"][0] < 1e-20


# ------------------------------------------------------ dual clip (second clip for negative advantages)

def test_dual_clip_hand_worked_table():
    """term = max(min(r a, clip(r) a), c a) for a < 0; untouched for a >= 0.  c = 3, bounds 0.8 / 1.28."""
    v = 4
    z = np.zeros((6, v))
    y = np.zeros(6, dtype=int)
    base = -math.log(v)                                   # logp of every token
    ratios = np.array([1.0, 2.0, 2.5, 4.0, 4.0, 0.5])
    a = np.array([-1.0, -1.0, -1.0, -1.0, 1.0, -1.0])
    logp_old = base - np.log(ratios)
    args = _identity_problem(z, y, logp_old, a)
    plain = O.loss_forward(*args)
    dual = O.loss_forward(*args, dual_clip=3.0)
    np.testing.assert_allclose(dual["ratio"], ratios, rtol=1e-14)
    # plain PPO-Clip terms: a<0: min(r a, clip(r) a) = -max(r, clip(r))
    np.testing.assert_allclose(plain["surrogate"], [-1.0, -2.0, -2.5, -4.0, 1.28, -0.8], rtol=1e-14)
    # with the second clip the term is bounded below by c a = -3
    np.testing.assert_allclose(dual["surrogate"], [-1.0, -2.0, -2.5, -3.0, 1.28, -0.8], rtol=1e-14)
    assert dual["unclipped"].tolist() == [True, True, True, False, False, False]
    assert plain["unclipped"].tolist() == [True, True, True, True, False, False]
    np.testing.assert_allclose(dual["coef"], [1 / 6, 2 / 6, 2.5 / 6, 0.0, 0.0, 0.0], rtol=1e-14)
    assert abs(dual["loss"] - (-(-1 - 2 - 2.5 - 3 + 1.28 - 0.8) / 6)) < 1e-14
    # a bound no ratio reaches changes nothing
    far = O.loss_forward(*args, dual_clip=100.0)
    assert far["loss"] == plain["loss"] and np.array_equal(far["coef"], plain["coef"])


def test_dual_clip_gradients_against_central_finite_differences():
    rng = np.random.default_rng(61)
    t, d, v = 6, 5, 9
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d)) * 0.5
    y = rng.integers(0, v, t)
    cu, a = [0, 3, 6], np.array([-0.9, 1.1])
    base = O.loss_forward(h, w, y, np.zeros(t), None, cu, a)
    # response 0 (a<0): ratios 1.1 (inside), 2.6 (beyond c = 2: constant term), 0.6 (first clip);
    # response 1 (a>0): 1.1, 2.6 (clipped above), 0.9
    logp_old = base["logp"] - np.log([1.1, 2.6, 0.6, 1.1, 2.6, 0.9])
    fwd = O.loss_forward(h, w, y, logp_old, None, cu, a, dual_clip=2.0)
    assert fwd["unclipped"].tolist() == [True, False, False, True, False, True]
    dh, dw = O.loss_backward(h, w, y, fwd["lse"], fwd["coef"])
    step = 1e-6
    for arr, grad in ((h, dh), (w, dw)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            keep = arr[idx]
            arr[idx] = keep + step
            up = O.loss_forward(h, w, y, logp_old, None, cu, a, dual_clip=2.0)["loss"]
            arr[idx] = keep - step
            dn = O.loss_forward(h, w, y, logp_old, None, cu, a, dual_clip=2.0)["loss"]
            arr[idx] = keep
            num[idx] = (up - dn) / (2 * step)
        assert np.linalg.norm(num - grad) <= 1e-6 * np.linalg.norm(grad)
    # without the second clip token 1 would carry gradient
    assert O.loss_forward(h, w, y, logp_old, None, cu, a)["coef"][1] != 0.0 and fwd["coef"][1] == 0.0


def test_dual_clip_on_the_sequence_level_objective_and_in_the_diagnostics():
    rng = np.random.default_rng(62)
    t, d, v = 8, 4, 7
    h, w = rng.standard_normal((t, d)), rng.standard_normal((v, d)) * 0.5
    y = rng.integers(0, v, t)
    cu, a = [0, 4, 8], np.array([-1.0, -0.5])
    base = O.loss_forward(h, w, y, np.zeros(t), None, cu, a)
    shift = np.concatenate([np.full(4, math.log(3.0)), np.full(4, math.log(1.1))])
    logp_old = base["logp"] - shift                       # response ratios 3.0 and 1.1
    g = O.loss_forward(h, w, y, logp_old, None, cu, a, surrogate=O.SUR_GSPO, dual_clip=2.0)
    np.testing.assert_allclose(g["ratio"], np.repeat([3.0, 1.1], 4), rtol=1e-12)
    assert abs(g["loss"] - (-(2.0 * -1.0 + 1.1 * -0.5) / 2)) < 1e-12      # c a for the first, r a for the second
    assert np.all(g["coef"][:4] == 0.0) and np.all(g["coef"][4:] != 0.0)
    # diagnostics: the share of stopped tokens counts the second clip and equals the zero-coef share
    tok = O.loss_forward(h, w, y, logp_old, None, cu, a, dual_clip=2.0)
    st = O.loss_stats(tok["logp"], logp_old, None, cu, a, dual_clip=2.0)
    assert abs(st[2] - (tok["coef"] == 0.0).mean()) < 1e-15 and st[2] == 0.5
    assert O.loss_stats(tok["logp"], logp_old, None, cu, a)[2] == 0.0
