"""GPU parity of the tracker, advantage and sampling kernels against the CPU oracle.

Tolerances: tracker / advantage / normalisation values 1e-5 relative in fp32 (plus an
absolute floor of 1e-6 where values pass through zero).  Sampling: the weights the library
emits are held to the float64 definition (Eq. "sampling_coef") at 1e-5 relative, and the
sampled ids must equal, bit for bit, what the oracle's selector draws from those same
weights and uniforms; a call that does not emit the weights must return the same ids.
"""

import math

import numpy as np
import pytest

from oracle import spo_oracle as O
from paper_2509_13232_b200 import inputs
from tests.helpers import dev, status_word, ws_bytes

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-6


def B():
    from paper_2509_13232_b200 import binding
    return binding


def gpu_init(v0, params):
    import torch
    ab = torch.empty((len(v0), 2), dtype=torch.float32, device="cuda")
    B().spo_tracker_init(ab, dev(v0), params)
    return ab


def gpu_sample(ab_t, u, batch, params, want_w=True):
    import torch
    n = ab_t.shape[0]
    ids = torch.full((batch,), -7, dtype=torch.int32, device="cuda")
    w = torch.empty(n, dtype=torch.float32, device="cuda") if want_w else None
    st = status_word()
    ws = ws_bytes(B().WS_SAMPLE, N=n, M=len(u))
    B().spo_sample_prompts(ab_t, dev(u), batch, ids, w, ws, params, st)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), (None if w is None else w.cpu().numpy()), int(st[0].item())


def check_draw(ab, u, batch, params, also_without_weights=True):
    """Draw on the GPU with the weights emitted; hold the weights to the float64 definition and the
    ids to the oracle's selector fed with those weights.  Returns (ids, weights, status)."""
    ab_t = dev(ab)
    ids, w, st = gpu_sample(ab_t, u, batch, params, want_w=True)
    want_w = O.sampling_weights(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64),
                                float(np.float32(params.eps_explore)))
    np.testing.assert_allclose(w, want_w, rtol=RTOL)
    np.testing.assert_array_equal(ids, O.sample_prompts(w, u, batch))
    if also_without_weights:
        ids2, _, st2 = gpu_sample(ab_t, u, batch, params, want_w=False)
        np.testing.assert_array_equal(ids2, ids)
        assert st2 == st
    return ids, w, st


def gpu_advantages(ab_t, ids, r, params, want_raw=True):
    import torch
    b = len(ids)
    a_raw = torch.empty(b, dtype=torch.float32, device="cuda") if want_raw else None
    a_norm = torch.empty(b, dtype=torch.float32, device="cuda")
    stats = torch.zeros(8, dtype=torch.float32, device="cuda")
    st = status_word()
    ws = ws_bytes(B().WS_ADVANTAGES, B=b)
    B().spo_advantages(ab_t, dev(ids), dev(r), a_raw, a_norm, stats, ws, params, st)
    torch.cuda.synchronize()
    return (None if a_raw is None else a_raw.cpu().numpy()), a_norm.cpu().numpy(), stats.cpu().numpy(), int(st[0].item())


def gpu_update(ab_t, ids, r, kl, is_table, params):
    import torch
    st = status_word()
    B().spo_tracker_update(ab_t, dev(ids), dev(r), dev(kl), is_table, params, st)
    torch.cuda.synchronize()
    return int(st[0].item())


def test_cfg1_tracker_step_matches_oracle():
    """Tiny step: Algorithm 2 init, sampling, advantage (pre-update), update, normalisation."""
    tb, _ = inputs.cfg1_tiny()
    p = B().default_params()
    ab_t = gpu_init(tb.v0, p)
    a0, b0 = O.tracker_init(tb.v0, 0.875)
    ab = ab_t.cpu().numpy()
    np.testing.assert_allclose(ab[:, 0], a0, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(ab[:, 1], b0, rtol=RTOL, atol=ATOL)
    assert np.allclose(ab.sum(axis=1), 8.0)
    # sampling: all 16 of 16 -> a permutation, bit-exact
    ids, w, st = check_draw(ab, tb.uniforms, 16, p)
    assert st == 0
    np.testing.assert_allclose(w, O.sampling_weights(a0, b0, float(np.float32(p.eps_explore))), rtol=RTOL)
    assert sorted(ids.tolist()) == list(range(16))
    # advantage before the update, then the update
    a_raw, a_norm, stats, st = gpu_advantages(ab_t, tb.ids, tb.rewards, p)
    assert st == 0
    want_raw = O.raw_advantage(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64), tb.ids, tb.rewards)
    want_norm, mu, sigma = O.normalise_advantages(want_raw, 0, float(np.float32(p.norm_eps)))
    np.testing.assert_allclose(a_raw, want_raw, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(a_norm, want_norm, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(stats[:3], [mu, sigma, 16], rtol=RTOL, atol=ATOL)
    assert gpu_update(ab_t, tb.ids, tb.rewards, tb.kl, 0, p) == 0
    a1, b1 = O.tracker_update(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64), tb.ids, tb.rewards,
                              tb.kl.astype(np.float64), float(np.float32(p.d_half)))
    ab1 = ab_t.cpu().numpy()
    np.testing.assert_allclose(ab1[:, 0], a1, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(ab1[:, 1], b1, rtol=RTOL, atol=ATOL)


@pytest.fixture(scope="module")
def cfg2():
    return inputs.tracker_batch(2, 1_000_000, 4096, 8192)


def test_cfg2_advantages_and_update_at_scale(cfg2):
    tb = cfg2
    p = B().default_params()
    ab_t = dev(tb.ab)
    a64, b64 = tb.ab[:, 0].astype(np.float64), tb.ab[:, 1].astype(np.float64)
    a_raw, a_norm, stats, st = gpu_advantages(ab_t, tb.ids, tb.rewards, p)
    assert st == 0
    want_raw = O.raw_advantage(a64, b64, tb.ids, tb.rewards)
    want_norm, mu, sigma = O.normalise_advantages(want_raw, 0, float(np.float32(p.norm_eps)))
    np.testing.assert_allclose(a_raw, want_raw, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(a_norm, want_norm, rtol=RTOL, atol=2e-6)
    np.testing.assert_allclose(stats[:2], [mu, sigma], rtol=RTOL, atol=ATOL)
    # per-prompt divergence table gathered by id
    assert gpu_update(ab_t, tb.ids, tb.rewards, tb.kl_table, 1, p) == 0
    a1, b1 = O.tracker_update(a64, b64, tb.ids, tb.rewards, tb.kl.astype(np.float64), float(np.float32(p.d_half)))
    ab1 = ab_t.cpu().numpy()
    np.testing.assert_allclose(ab1[:, 0], a1, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(ab1[:, 1], b1, rtol=RTOL, atol=ATOL)
    # all three branches of the clamp occur in this workload
    rho = O.forgetting_factor(tb.kl.astype(np.float64), float(np.float32(p.d_half)))
    assert (rho == 0.875).any() and (rho == 0.96).any() and ((rho > 0.875) & (rho < 0.96)).any()


def test_cfg2_sampling_bit_exact(cfg2):
    tb = cfg2
    p = B().default_params()
    ids, w, st = check_draw(tb.ab, tb.uniforms, 4096, p)
    assert st == 0
    assert len(set(ids.tolist())) == 4096


@pytest.mark.parametrize("n,m,b", [(1, 4, 1), (5, 64, 5), (2047, 300, 100), (2049, 128, 64), (70001, 4096, 2048)])
def test_sampling_ragged_sizes_and_repeats(n, m, b):
    """Odd table sizes (tile tails), heavy repetition (small N), no weight output."""
    rng = np.random.default_rng(100 + n)
    ab = rng.uniform(0.0, 12.0, (n, 2)).astype(np.float32)
    if n > 4:
        ab[1] = 0.0            # empty entry -> v = 0.5
        ab[2, 0] = 0.0         # v = 0 -> weight eps
    u = inputs.uniforms_f32(rng, m)
    p = B().default_params()
    ids, _, st = check_draw(ab, u, b, p)
    assert st == 0


def test_sampling_reports_exhausted_uniforms():
    ab = np.ones((4, 2), dtype=np.float32)
    u = np.array([0.1, 0.1, 0.1, 0.1], dtype=np.float32)       # always the same prompt
    ids, _, st = gpu_sample(dev(ab), u, 3, B().default_params())
    assert st & B().DEV_UNIFORMS_EXHAUSTED
    assert ids[0] == 0 and (ids[1:] == -1).all()


def test_advantages_large_batch_two_pass_path():
    rng = np.random.default_rng(7)
    n, b = 300_000, 200_000
    ab = rng.uniform(0.1, 12.0, (n, 2)).astype(np.float32)
    ids = rng.permutation(n)[:b].astype(np.int32)
    r = (rng.random(b) < 0.4).astype(np.float32)
    for ddof, want_raw in ((0, True), (1, False)):
        p = B().default_params(norm_ddof=ddof)
        a_raw, a_norm, stats, st = gpu_advantages(dev(ab), ids, r, p, want_raw=want_raw)
        want = O.raw_advantage(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64), ids, r)
        want_norm, mu, sigma = O.normalise_advantages(want, ddof, float(np.float32(p.norm_eps)))
        assert st == 0
        if want_raw:
            np.testing.assert_allclose(a_raw, want, rtol=RTOL, atol=ATOL)
        np.testing.assert_allclose(a_norm, want_norm, rtol=RTOL, atol=2e-6)
        np.testing.assert_allclose(stats[:2], [mu, sigma], rtol=RTOL, atol=ATOL)


def test_advantages_degenerate_batches():
    p = B().default_params()
    ab = np.array([[2.0, 2.0], [0.0, 0.0], [0.0, 4.0]], dtype=np.float32)
    # one entry: normalised advantage is zero
    _, a_norm, _, _ = gpu_advantages(dev(ab), np.array([0], np.int32), np.array([1.0], np.float32), p)
    assert a_norm[0] == 0.0
    # all-equal advantages -> zeros; empty entry estimates 0.5; zero table -> A = r
    a_raw, a_norm, stats, _ = gpu_advantages(dev(ab), np.array([0, 1], np.int32), np.array([1.0, 1.0], np.float32), p)
    np.testing.assert_array_equal(a_raw, [0.5, 0.5])
    np.testing.assert_array_equal(a_norm, [0.0, 0.0])
    a_raw, _, _, _ = gpu_advantages(dev(ab), np.array([2], np.int32), np.array([1.0], np.float32), p)
    assert a_raw[0] == 1.0
    # an id outside the table is reported, not dereferenced
    _, _, _, st = gpu_advantages(dev(ab), np.array([0, 9], np.int32), np.array([1.0, 0.0], np.float32), p)
    assert st & B().DEV_ID_OUT_OF_RANGE


def test_update_flags_bad_entries_and_leaves_them_untouched():
    p = B().default_params()
    ab = np.array([[2.0, 2.0], [1.0, 3.0], [3.0, 1.0]], dtype=np.float32)
    ab_t = dev(ab)
    st = gpu_update(ab_t, np.array([0, 5, 2], np.int32), np.array([1.0, 1.0, 0.0], np.float32),
                    np.array([0.01, 0.01, np.nan], np.float32), 0, p)
    assert st & B().DEV_ID_OUT_OF_RANGE and st & B().DEV_NONFINITE
    out = ab_t.cpu().numpy()
    np.testing.assert_array_equal(out[1:], ab[1:])
    a1, b1 = O.tracker_update([2.0], [2.0], [0], [1.0], [np.float64(np.float32(0.01))], float(np.float32(p.d_half)))
    np.testing.assert_allclose(out[0], [a1[0], b1[0]], rtol=RTOL)


def test_sampling_single_prompt_table_and_full_draw():
    p = B().default_params()
    ids, w, st = check_draw(np.array([[3.0, 1.0]], np.float32), np.array([0.7, 0.2], np.float32), 1, p)
    assert st == 0 and ids.tolist() == [0]
    assert abs(float(w[0]) - (math.sqrt(0.75 * 0.25) + 0.05)) < 1e-6
    # B = M = N: every uniform must land on a new prompt, else the call reports exhaustion
    n = 8
    ab = np.full((n, 2), 2.0, dtype=np.float32)
    u = ((np.arange(n) + 0.5) / n).astype(np.float32)
    ids, _, st = gpu_sample(dev(ab), u, n, p)
    assert st == 0 and ids.tolist() == list(range(n))


def test_sampling_flags_bad_table_entries_and_zero_total_weight():
    p = B().default_params()
    ab = np.array([[2.0, 2.0], [-1.0, 2.0], [np.nan, 1.0], [1.0, 3.0]], dtype=np.float32)
    u = inputs.uniforms_f32(np.random.default_rng(3), 64)
    ids, w, st = gpu_sample(dev(ab), u, 2, p)
    assert st & B().DEV_NONFINITE
    assert w[1] == 0.0 and w[2] == 0.0 and set(ids.tolist()) == {0, 3}
    p0 = B().default_params(eps_explore=0.0)
    dead = np.array([[0.0, 5.0], [4.0, 0.0]], dtype=np.float32)      # v = 0 and v = 1: weight eps = 0
    ids, _, st = gpu_sample(dev(dead), u, 1, p0)
    assert st & B().DEV_ZERO_TOTAL_WEIGHT and ids[0] == -1


def test_sampling_across_super_tile_boundaries():
    """A table larger than one second-level group (1024 tiles of 2048 prompts)."""
    n = 2048 * 1024 * 2 + 777
    rng = np.random.default_rng(11)
    ab = rng.uniform(0.0, 9.0, (n, 2)).astype(np.float32)
    u = inputs.uniforms_f32(rng, 512)
    p = B().default_params()
    ids, _, st = check_draw(ab, u, 256, p)
    assert st == 0


def test_fractional_rewards_update_and_advantages():
    """Rewards anywhere in [0,1] (the paper's EMA remark for general rewards) go through the same kernels."""
    rng = np.random.default_rng(31)
    n, b = 50_000, 20_000
    ab = rng.uniform(0.1, 12.0, (n, 2)).astype(np.float32)
    ids = rng.permutation(n)[:b].astype(np.int32)
    r = rng.uniform(0.0, 1.0, b).astype(np.float32)
    kl = rng.lognormal(-4, 1, b).astype(np.float32)
    p = B().default_params()
    ab_t = dev(ab)
    a_raw, a_norm, stats, st = gpu_advantages(ab_t, ids, r, p)
    a64, b64 = ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64)
    want_raw = O.raw_advantage(a64, b64, ids, r)
    want_norm, mu, sigma = O.normalise_advantages(want_raw, 0, float(np.float32(p.norm_eps)))
    assert st == 0
    np.testing.assert_allclose(a_raw, want_raw, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(a_norm, want_norm, rtol=RTOL, atol=2e-6)
    assert gpu_update(ab_t, ids, r, kl, 0, p) == 0
    a1, b1 = O.tracker_update(a64, b64, ids, r, kl.astype(np.float64), float(np.float32(p.d_half)))
    out = ab_t.cpu().numpy()
    np.testing.assert_allclose(out[:, 0], a1, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(out[:, 1], b1, rtol=RTOL, atol=ATOL)


@pytest.mark.parametrize("n,b,g", [(64, 512, 8), (5000, 16384, 8), (3, 100, 40), (1000, 65536, 70)])
def test_batch_spo_repeated_ids(n, b, g):
    """Every prompt appears about g times; shared pre-update baseline, updates composed in batch order."""
    import torch
    rng = np.random.default_rng(200 + n)
    ab = rng.uniform(0.1, 12.0, (n, 2)).astype(np.float32)
    ids = rng.integers(0, n, b).astype(np.int32)
    r = (rng.random(b) < 0.5).astype(np.float32)
    kl = rng.lognormal(-4, 1, b).astype(np.float32)
    p = B().default_params()
    ab_t = dev(ab)
    a_raw, a_norm, _, st = gpu_advantages(ab_t, ids, r, p)
    a64, b64 = ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64)
    want_raw = O.raw_advantage(a64, b64, ids, r)
    np.testing.assert_allclose(a_raw, want_raw, rtol=RTOL, atol=ATOL)
    ws = ws_bytes(B().WS_UPDATE_REPEATS, B=b)
    stw = status_word()
    B().spo_tracker_update_repeats(ab_t, dev(ids), dev(r), dev(kl), 0, ws, p, stw)
    torch.cuda.synchronize()
    assert int(stw[0].item()) == 0
    a1, b1 = O.tracker_update(a64, b64, ids, r, kl.astype(np.float64), float(np.float32(p.d_half)))
    out = ab_t.cpu().numpy()
    # up to g roundings compose per prompt: tolerance scaled accordingly
    np.testing.assert_allclose(out[:, 0], a1, rtol=RTOL * 4, atol=ATOL * 4)
    np.testing.assert_allclose(out[:, 1], b1, rtol=RTOL * 4, atol=ATOL * 4)
    # bit-identical on a second run from the same start: no dependence on scheduling
    ab_t2 = dev(ab)
    B().spo_tracker_update_repeats(ab_t2, dev(ids), dev(r), dev(kl), 0, ws, p, stw)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(ab_t2.cpu().numpy(), out)


def test_batch_spo_update_skips_bad_entries():
    import torch
    p = B().default_params()
    ab = np.array([[2.0, 2.0], [1.0, 3.0]], dtype=np.float32)
    ab_t = dev(ab)
    ids = np.array([0, 7, 0, 1], np.int32)
    r = np.array([1.0, 1.0, np.nan, 0.0], np.float32)
    kl = np.array([0.01, 0.01, 0.01, 0.01], np.float32)
    st = status_word()
    B().spo_tracker_update_repeats(ab_t, dev(ids), dev(r), dev(kl), 0, ws_bytes(B().WS_UPDATE_REPEATS, B=4), p, st)
    torch.cuda.synchronize()
    word = int(st[0].item())
    assert word & B().DEV_ID_OUT_OF_RANGE and word & B().DEV_NONFINITE
    a1, b1 = O.tracker_update([2.0, 1.0], [2.0, 3.0], [0, 1], [1.0, 0.0], [np.float64(np.float32(0.01))] * 2,
                              float(np.float32(p.d_half)))
    np.testing.assert_allclose(ab_t.cpu().numpy(), np.stack([a1, b1], 1), rtol=RTOL)


@pytest.mark.parametrize("n", [1, 2047, 4097])
def test_sampling_weight_output_for_odd_table_sizes(n):
    rng = np.random.default_rng(300 + n)
    ab = rng.uniform(0.0, 12.0, (n, 2)).astype(np.float32)
    u = inputs.uniforms_f32(rng, 32)
    p = B().default_params()
    ids, w, st = check_draw(ab, u, 1, p)
    assert st == 0 and w.shape == (n,)


def test_sampling_at_the_maximum_number_of_uniforms():
    """M = 2^20 draws (the documented limit) with many repeats; ids still bit-exact and in order."""
    n, m, b = 3_000_000, 1 << 20, 500_000
    rng = np.random.default_rng(404)
    ab = rng.uniform(0.0, 12.0, (n, 2)).astype(np.float32)
    u = inputs.uniforms_f32(rng, m)
    p = B().default_params()
    ids, _, st = check_draw(ab, u, b, p)
    assert st == 0
    assert len(set(ids.tolist())) == b


def test_sampling_weights_over_thirty_decades_of_table_magnitudes():
    """Common entries, empty entries, a zero parameter, tiny and huge magnitudes: every weight
    within 1e-5 of the float64 definition, and the draw made from them is the oracle's."""
    rng = np.random.default_rng(41)
    special = np.array([[0, 0], [0, 5], [5, 0], [1e-30, 1], [1, 1e-38], [1e-20, 1e-20], [1e25, 1e25],
                        [3e5, 7e5], [2.0 ** -21, 2.0 ** -21], [1e-39, 1], [8, 8], [0.875, 7.125],
                        [1e18, 3e18], [1e-19, 4e-19]], dtype=np.float32)
    ab = np.concatenate([special, rng.uniform(0.0, 25.0, (3000, 2)).astype(np.float32),
                         (10.0 ** rng.uniform(-12, 12, (3000, 2))).astype(np.float32)])
    ab = ab[rng.permutation(len(ab))]
    p = B().default_params()
    u = inputs.uniforms_f32(rng, 600)
    ids, w, st = check_draw(ab, u, 300, p)
    assert st == 0
    eps = np.float32(p.eps_explore)
    assert w.min() >= eps and w.max() <= np.float32(0.5) + eps          # the range Eq. "sampling_coef" gives


def gpu_advantages_update(ab_t, ids, r, kl, is_table, params, want_raw=True):
    import torch
    b = len(ids)
    a_raw = torch.full((b,), float("nan"), dtype=torch.float32, device="cuda") if want_raw else None
    a_norm = torch.full((b,), float("nan"), dtype=torch.float32, device="cuda")
    stats = torch.zeros(8, dtype=torch.float32, device="cuda")
    st = status_word()
    ws = ws_bytes(B().WS_ADVANTAGES, B=b)
    B().spo_advantages_update(ab_t, dev(ids), dev(r), dev(kl), is_table, a_raw, a_norm, stats, ws, params, st)
    torch.cuda.synchronize()
    return (None if a_raw is None else a_raw.cpu().numpy()), a_norm.cpu().numpy(), stats.cpu().numpy(), int(st[0].item())


@pytest.mark.parametrize("n,b,is_table", [(1_000_000, 4096, 1), (300_000, 200_000, 0), (50, 7, 0), (40_000, 8193, 1)])
def test_fused_advantage_and_update_equals_the_two_steps_in_the_papers_order(n, b, is_table):
    """One pass over the batch's entries: the advantage is formed from the estimate as read
    (before this batch's update), then the entry is updated -- Algorithm 1's order.  Single-block
    and two-pass sizes, divergences per entry and per prompt."""
    rng = np.random.default_rng(900 + b)
    ab = rng.uniform(0.1, 12.0, (n, 2)).astype(np.float32)
    ab[rng.integers(0, n, max(1, n // 50))] = 0.0                  # some empty entries (v = 0.5, then v = r)
    ids = rng.permutation(n)[:b].astype(np.int32)
    a64, b64 = ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64)
    v = O.value_estimate(a64, b64)
    r = (rng.random(b) < v[ids]).astype(np.float32)
    kl_table = rng.lognormal(-4, 1, n).astype(np.float32)
    kl = kl_table[ids]
    p = B().default_params(norm_ddof=1 if b == 8193 else 0)
    ab_t = dev(ab)
    a_raw, a_norm, stats, st = gpu_advantages_update(ab_t, ids, r, kl_table if is_table else kl, is_table, p,
                                                     want_raw=(b != 8193))
    assert st == 0
    want_raw = O.raw_advantage(a64, b64, ids, r)
    want_norm, mu, sigma = O.normalise_advantages(want_raw, p.norm_ddof, float(np.float32(p.norm_eps)))
    if a_raw is not None:
        np.testing.assert_allclose(a_raw, want_raw, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(a_norm, want_norm, rtol=RTOL, atol=2e-6)
    np.testing.assert_allclose(stats[:3], [mu, sigma, b], rtol=RTOL, atol=ATOL)
    a1, b1 = O.tracker_update(a64, b64, ids, r, kl.astype(np.float64), float(np.float32(p.d_half)))
    out = ab_t.cpu().numpy()
    np.testing.assert_allclose(out[:, 0], a1, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(out[:, 1], b1, rtol=RTOL, atol=ATOL)
    # and it is the same as the two separate calls
    ab_t2 = dev(ab)
    a_raw2, a_norm2, stats2, _ = gpu_advantages(ab_t2, ids, r, p)
    gpu_update(ab_t2, ids, r, kl_table if is_table else kl, is_table, p)
    np.testing.assert_array_equal(a_norm2, a_norm)
    np.testing.assert_array_equal(stats2, stats)
    np.testing.assert_array_equal(ab_t2.cpu().numpy(), out)


def test_fused_advantage_and_update_skips_bad_elements():
    p = B().default_params()
    ab = np.array([[2.0, 2.0], [1.0, 3.0], [3.0, 1.0], [-1.0, 2.0], [4.0, 4.0]], dtype=np.float32)
    ab_t = dev(ab)
    ids = np.array([0, 9, 2, 3, 4, 1], np.int32)
    r = np.array([1.0, 1.0, np.nan, 1.0, 0.0, 1.0], np.float32)
    kl = np.array([0.01, 0.01, 0.01, 0.01, np.nan, 0.02], np.float32)
    a_raw, _, _, st = gpu_advantages_update(ab_t, ids, r, kl, 0, p)
    assert st & B().DEV_ID_OUT_OF_RANGE and st & B().DEV_NONFINITE
    # bad id, NaN reward, negative entry: A = 0, entry untouched; NaN divergence: A defined, entry untouched
    np.testing.assert_allclose(a_raw, [0.5, 0.0, 0.0, 0.0, -0.5, 0.75], rtol=RTOL)
    out = ab_t.cpu().numpy()
    np.testing.assert_array_equal(out[2:5], ab[2:5])
    a1, b1 = O.tracker_update(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64), [0, 1], [1.0, 1.0],
                              [np.float64(np.float32(0.01)), np.float64(np.float32(0.02))], float(np.float32(p.d_half)))
    np.testing.assert_allclose(out[:2], np.stack([a1[:2], b1[:2]], 1), rtol=RTOL)


def test_near_zero_advantage_counts():
    """Sec. 4 tracks the share of raw advantages with |A| <= tau at tau = 1e-4 and 0.02."""
    rng = np.random.default_rng(77)
    p = B().default_params()
    # hand case: estimates 1, 0.99, 0.5, 0 against rewards 1, 1, 1, 0 -> |A| = 0, 0.01, 0.5, 0
    ab = np.array([[8.0, 0.0], [7.92, 0.08], [4.0, 4.0], [0.0, 8.0]], dtype=np.float32)
    _, _, stats, st = gpu_advantages(dev(ab), np.arange(4, dtype=np.int32), np.array([1, 1, 1, 0], np.float32), p)
    assert st == 0 and stats[4] == 2.0 and stats[5] == 3.0 and stats[6] == 0.0 and stats[7] == 0.0
    # both code paths, against the oracle's counts, with tolerances set by the caller
    n = 200_000
    v = rng.beta(0.3, 0.3, n)                                      # many prompts nearly mastered or hopeless
    ab = np.stack([v * 16.0, (1.0 - v) * 16.0], 1).astype(np.float32)
    for b in (4096, 150_000):
        ids = rng.permutation(n)[:b].astype(np.int32)
        est = O.value_estimate(ab[ids, 0].astype(np.float64), ab[ids, 1].astype(np.float64))
        r = (rng.random(b) < est).astype(np.float32)
        for taus in ((1e-4, 0.02), (0.005, 0.1)):
            pp = B().default_params(near_zero_tau_lo=taus[0], near_zero_tau_hi=taus[1])
            a_raw, _, stats, st = gpu_advantages(dev(ab), ids, r, pp)
            f32_taus = (float(np.float32(taus[0])), float(np.float32(taus[1])))
            want = O.near_zero_counts(a_raw, f32_taus)             # the same fp32 advantages, so the counts are exact
            assert st == 0 and [int(stats[4]), int(stats[5])] == want and want[1] > want[0] > 0
            loose = O.near_zero_counts(O.raw_advantage(ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64), ids, r),
                                       f32_taus)
            assert abs(loose[1] - want[1]) <= 1 + b // 10_000        # float64 advantages: ties at tau may differ


def test_update_from_an_empty_entry_gives_the_first_reward():
    """The start without offline initialisation (appendix ablation): an entry (0, 0) estimates 0.5 and
    after its first update the estimate is the reward itself, whatever the divergence."""
    p = B().default_params()
    n = 64
    ab = np.zeros((n, 2), dtype=np.float32)
    ab[1::2] = [2.0, 6.0]
    ids = np.arange(0, n, 2, dtype=np.int32)                      # the empty entries
    rng = np.random.default_rng(5)
    r = rng.uniform(0, 1, len(ids)).astype(np.float32)
    r[:4] = [0.0, 1.0, 1.0, 0.0]
    kl = rng.lognormal(-4, 1, len(ids)).astype(np.float32)
    for fused in (False, True):
        ab_t = dev(ab)
        if fused:
            a_raw, _, _, st = gpu_advantages_update(ab_t, ids, r, kl, 0, p)
        else:
            a_raw, _, _, st = gpu_advantages(ab_t, ids, r, p)
            st |= gpu_update(ab_t, ids, r, kl, 0, p)
        assert st == 0
        np.testing.assert_allclose(a_raw, r - 0.5, rtol=RTOL, atol=ATOL)
        out = ab_t.cpu().numpy()
        a1, b1 = O.tracker_update(np.zeros(n), np.zeros(n), ids, r, kl.astype(np.float64), float(np.float32(p.d_half)))
        np.testing.assert_allclose(out[ids, 0], a1[ids], rtol=RTOL, atol=ATOL)
        np.testing.assert_allclose(out[ids, 1], b1[ids], rtol=RTOL, atol=ATOL)
        np.testing.assert_allclose(O.value_estimate(out[ids, 0], out[ids, 1]), r, rtol=RTOL, atol=ATOL)
        np.testing.assert_array_equal(out[1::2], ab[1::2])


def test_advantages_flag_bad_table_entries_and_rewards():
    p = B().default_params()
    ab = np.array([[2.0, 2.0], [np.inf, 1.0], [1.0, -3.0], [3.0, 1.0]], dtype=np.float32)
    a_raw, _, _, st = gpu_advantages(dev(ab), np.array([0, 1, 2, 3], np.int32), np.array([1, 1, 1, np.inf], np.float32), p)
    assert st & B().DEV_NONFINITE and not st & B().DEV_ID_OUT_OF_RANGE
    np.testing.assert_array_equal(a_raw, [0.5, 0.0, 0.0, 0.0])
