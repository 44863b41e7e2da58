"""GPU parity of the fused loss forward / backward against the CPU oracle.

Tolerances (bf16 inputs, fp32 accumulation): loss and per-token log-probs within 2e-3
absolute; gradients within 1e-2 relative Frobenius error.  The fp32 path is held to
1e-4 absolute / 1e-4 relative Frobenius.
"""

import numpy as np
import pytest

from oracle import spo_oracle as O
from paper_2509_13232_b200 import inputs
from tests.helpers import oracle_loss, rel_fro, run_loss

pytestmark = pytest.mark.gpu


def check(lb, got, want, abs_tol, fro_tol):
    assert got["status"] == 0
    assert abs(got["loss"] - want["loss"]) <= abs_tol
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=abs_tol)
    np.testing.assert_allclose(got["lse"], want["lse"], rtol=0, atol=abs_tol)
    assert rel_fro(got["coef"], want["coef"]) <= fro_tol
    if got["seq_sums"] is not None:
        scale = np.maximum(1.0, want["seq_sums"][:, 2:3])
        np.testing.assert_allclose(got["seq_sums"] / scale, want["seq_sums"] / scale, rtol=0, atol=abs_tol)
    assert rel_fro(got["dH"], want["dH"]) <= fro_tol
    assert rel_fro(got["dW"], want["dW"]) <= fro_tol


def test_cfg1_tiny_fp32_full_parity():
    tb, lb = inputs.cfg1_tiny()
    # advantages of the tiny step come from the oracle's own tracker pieces
    a0, b0 = O.tracker_init(tb.v0, 0.875)
    a_norm, _, _ = O.normalise_advantages(O.raw_advantage(a0, b0, tb.ids, tb.rewards))
    lb.a_norm = a_norm.astype(np.float32)
    got = run_loss(lb)
    want = oracle_loss(lb)
    check(lb, got, want, 1e-4, 1e-4)
    assert abs(want["n_tok"] - lb.h.shape[0]) == 0


def _clip_batch(cfg, lengths, d, v, bf16, w_std=0.05):
    """Old log-probs far enough from the new ones that all four (sign x side) clip branches occur."""
    rng = np.random.default_rng(cfg)
    a = rng.standard_normal(len(lengths)).astype(np.float32)
    a[0] = 0.0
    return inputs.loss_batch(cfg, lengths, d, v, w_std, bf16, 0.3, target="softmax", mask_p=0.15, a_norm=a)


def test_fp32_clip_branches_mask_and_grad_scale():
    lb = _clip_batch(11, [5, 17, 1, 30, 9], 32, 257, False)
    got = run_loss(lb, grad_loss=0.37, dh_bf16=False)
    want = oracle_loss(lb, grad_loss=0.37)
    assert 0.05 < want["unclipped"].mean() < 0.95
    check(lb, got, want, 1e-4, 1e-4)
    masked = lb.mask == 0
    assert masked.any() and np.all(got["dH"][masked] == 0.0)


def test_fp32_dw_accumulate_and_no_mask():
    lb = inputs.loss_batch(12, [7, 8], 16, 50, 0.1, False, 0.05)
    init = np.random.default_rng(1).standard_normal((50, 16)).astype(np.float32)
    got = run_loss(lb, dw_init=init, mask_none=True)
    want = oracle_loss(lb, mask_none=True)
    assert rel_fro(got["dW"] - init, want["dW"]) <= 1e-4
    assert abs(got["loss"] - want["loss"]) <= 1e-4


BF16_CASES = [
    # name, lengths, d, V
    ("one_tile_ragged", [40, 60], 64, 200),
    ("tails_everywhere", [100, 1, 200, 29], 128, 1000),
    ("short_k_many_vocab_tiles", [300, 500, 240], 192, 5000),
    ("several_token_tiles", [700, 900, 404], 256, 2304),
]


@pytest.mark.parametrize("name,lengths,d,v", BF16_CASES, ids=[c[0] for c in BF16_CASES])
def test_bf16_parity_small_shapes(name, lengths, d, v):
    lb = _clip_batch(20 + len(lengths) + d, lengths, d, v, True, w_std=0.05)
    got = run_loss(lb, grad_loss=1.0)
    want = oracle_loss(lb)
    assert 0.02 < 1.0 - want["unclipped"].mean()
    check(lb, got, want, 2e-3, 1e-2)


def test_bf16_fp32_dh_output_and_dw_accumulate_across_chunks():
    """More token rows than one backward chunk holds: dW is accumulated chunk by chunk."""
    lengths = [2000, 1500, 1100, 97]
    lb = inputs.loss_batch(31, lengths, 128, 1200, 0.05, True, 0.05, target="softmax")
    init = np.full((1200, 128), 0.25, dtype=np.float32)
    got = run_loss(lb, dh_bf16=False, dw_init=init)
    want = oracle_loss(lb)
    assert got["status"] == 0
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)
    assert rel_fro(got["dH"], want["dH"]) <= 1e-2
    assert rel_fro(got["dW"] - init, want["dW"]) <= 1e-2


def test_bf16_uniform_logits_and_bad_target():
    """W = 0 gives logp = -log V exactly; a target outside the vocabulary is flagged."""
    lb = inputs.loss_batch(32, [50, 78], 64, 300, 0.05, True, 0.05, target="uniform")
    lb.w[:] = 0.0
    got = run_loss(lb)
    np.testing.assert_allclose(got["logp"], -np.log(300.0), atol=1e-5)
    lb.y[3] = 300
    got = run_loss(lb)
    assert got["status"] & 1
    assert np.isneginf(got["logp"][3]) and got["coef"][3] == 0.0
    # a masked row may carry an ignore-index target: no gradient, no status bit
    lb.y[3] = -100
    lb.mask[3] = 0
    for one_pass in (False, True):
        got = run_loss(lb, one_pass=one_pass)
        assert got["status"] == 0 and got["coef"][3] == 0.0 and np.all(got["dH"][3] == 0.0)
        keep = np.arange(len(lb.y)) != 3
        np.testing.assert_allclose(got["logp"][keep], -np.log(300.0), atol=1e-5)


def test_empty_batch_is_a_no_op_with_zero_loss():
    """T = 0: loss 0, dW zeroed (or left alone when accumulating), nothing else touched."""
    import torch
    from paper_2509_13232_b200 import binding as B
    from tests.helpers import status_word, ws_bytes
    p = B.default_params()
    for dt, d, v in ((torch.bfloat16, 64, 300), (torch.float32, 16, 40)):
        H = torch.empty((0, d), dtype=dt, device="cuda")
        W = torch.randn((v, d), device="cuda").to(dt)
        z = lambda n, t=torch.float32: torch.zeros(max(n, 1), dtype=t, device="cuda")  # noqa: E731
        loss = torch.full((4,), 7.0, device="cuda")
        cu = torch.zeros(1, dtype=torch.int32, device="cuda")
        st = status_word()
        B.spo_loss_fwd(H, W, z(0, torch.int32), z(0), None, cu, z(0), loss, z(0), z(0), z(0), None,
                       ws_bytes(B.WS_LOSS_FWD, T=0, d=d, V=v, B=1), p, st)
        dW = torch.full((v, d), 3.0, device="cuda")
        dH = torch.empty((0, d), dtype=dt, device="cuda")
        B.spo_loss_bwd(H, W, z(0, torch.int32), z(0), z(0), 1.0, dH, dW, 0, ws_bytes(B.WS_LOSS_BWD, T=0, d=d, V=v), p, st)
        torch.cuda.synchronize()
        assert loss[0].item() == 0.0 and int(st[0].item()) == 0
        if dt == torch.bfloat16:
            assert float(dW.abs().max().item()) == 0.0


@pytest.mark.parametrize("bf16", [False, True])
def test_all_tokens_masked_gives_zero_loss_and_zero_gradients(bf16):
    lb = inputs.loss_batch(51, [20, 13], 64, 200, 0.05, bf16, 0.1)
    lb.mask[:] = 0
    got = run_loss(lb)
    want = oracle_loss(lb)
    assert want["loss"] == 0.0 and got["loss"] == 0.0 and got["status"] == 0
    assert np.all(got["coef"] == 0.0) and np.all(got["dH"] == 0.0) and np.all(got["dW"] == 0.0)
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)


@pytest.mark.parametrize("bf16", [False, True])
def test_single_token_and_empty_sequences(bf16):
    """One token row; and responses of length zero in the middle of the batch."""
    tol = (2e-3, 1e-2) if bf16 else (1e-4, 1e-4)
    one = inputs.loss_batch(52, [1], 64, 130, 0.05, bf16, 0.1)
    check(one, run_loss(one), oracle_loss(one), *tol)
    gaps = inputs.loss_batch(53, [5, 0, 0, 9, 0, 3], 64, 130, 0.05, bf16, 0.3,
                             a_norm=np.array([1.0, 9.0, -9.0, -0.7, 5.0, 0.4], dtype=np.float32))
    got, want = run_loss(gaps), oracle_loss(gaps)
    check(gaps, got, want, *tol)
    np.testing.assert_array_equal(got["seq_sums"][[1, 2, 4]], 0.0)


@pytest.mark.parametrize("v", [100, 512, 1024, 1025])
def test_bf16_vocabulary_edges(v):
    """Vocabulary below one tile, exactly one and two tiles, and one column over."""
    lb = _clip_batch(60 + v, [70, 61], 64, v, True)
    check(lb, run_loss(lb), oracle_loss(lb), 2e-3, 1e-2)


def test_bf16_targets_on_tile_and_half_boundaries():
    """Targets at the first/last column of accumulator halves and tiles are gathered correctly."""
    lb = inputs.loss_batch(70, [64], 64, 1200, 0.05, True, 0.05, target="uniform")
    edges = [0, 31, 32, 255, 256, 511, 512, 767, 768, 1023, 1024, 1199]
    lb.y[:len(edges)] = edges
    z = lb.h.astype(np.float64) @ lb.w.astype(np.float64).T
    from scipy.special import log_softmax
    lb.logp_old[:] = log_softmax(z, axis=1)[np.arange(64), lb.y].astype(np.float32)
    got, want = run_loss(lb), oracle_loss(lb)
    check(lb, got, want, 2e-3, 1e-2)
    np.testing.assert_allclose(want["ratio"], 1.0, atol=1e-6)


def test_bounded_wait_ends_in_a_status_bit_not_a_hang():
    """A barrier nobody signals: the wait gives up after its limit, the kernel returns, the context lives on."""
    import time
    import torch
    from paper_2509_13232_b200 import binding as B
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    end = torch.zeros(4, dtype=torch.int32, device="cuda")
    t0 = time.perf_counter()
    B.spo_selftest_bounded_wait(2000, end, st)          # 2 ms limit
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    assert int(st[0].item()) & B.DEV_TIMEOUT
    assert int(end[0].item()) == 1
    assert elapsed < 1.0
    # the device is still usable afterwards
    lb = inputs.loss_batch(80, [33], 64, 200, 0.05, True, 0.05)
    assert run_loss(lb)["status"] == 0


@pytest.mark.parametrize("bf16", [False, True])
def test_sequence_mean_aggregation(bf16):
    """Each response weighs the same whatever its length; fully masked and empty responses drop out."""
    from paper_2509_13232_b200 import binding as B
    params = B.default_params(agg_mode=B.AGG_SEQ_MEAN)
    lb = _clip_batch(90, [3, 40, 0, 17, 1, 9], 64, 333, bf16)
    lb.mask[3:43] = 0                                   # response 1 entirely masked
    lb.mask[50] = 0
    got = run_loss(lb, params=params, grad_loss=0.8)
    want = oracle_loss(lb, params=params, grad_loss=0.8)
    tol = (2e-3, 1e-2) if bf16 else (1e-4, 1e-4)
    check(lb, got, want, *tol)
    # and it differs from the token mean on this batch, so the switch is really exercised
    other = oracle_loss(lb, grad_loss=0.8)
    assert abs(other["loss"] - want["loss"]) > 1e-3
    for mask_none in (True,):
        got = run_loss(lb, params=params, mask_none=mask_none)
        want = oracle_loss(lb, params=params, mask_none=mask_none)
        check(lb, got, want, *tol)


def test_results_are_bitwise_reproducible():
    """Fixed reduction orders everywhere: two runs on the same inputs agree bit for bit
    (loss fold, split merge, chunked dW accumulation)."""
    lb = inputs.loss_batch(95, [2000, 1500, 1100, 97, 5300], 128, 1200, 0.05, True, 0.3, target="softmax", mask_p=0.1)
    a = run_loss(lb, grad_loss=0.9)
    b = run_loss(lb, grad_loss=0.9)
    assert a["loss"] == b["loss"]
    for k in ("logp", "lse", "coef", "dH", "dW", "seq_sums"):
        np.testing.assert_array_equal(a[k], b[k])


@pytest.mark.parametrize("dh_f32", [False, True])
def test_backward_over_active_rows_only(dh_f32):
    """40 % of the tokens masked (plus clipped ones): the row-compacted backward gives the oracle's gradients,
    zeros in the rows without gradient, and lists exactly the rows with coef != 0."""
    import torch
    from paper_2509_13232_b200 import binding as B
    from tests.helpers import dev, status_word, ws_bytes
    lb = _clip_batch(110, [900, 1300, 2, 700, 2500, 61], 128, 1500, True)
    rng = np.random.default_rng(3)
    lb.mask[:] = (rng.random(lb.mask.shape[0]) > 0.4).astype(np.uint8)
    lb.mask[900:2200] = 0                                # a whole response (tool output) masked
    want = oracle_loss(lb, grad_loss=0.7)
    p = B.default_params()
    H, W = dev(lb.h, torch.bfloat16), dev(lb.w, torch.bfloat16)
    T, d = H.shape
    V = W.shape[0]
    y = dev(lb.y)
    lse, coef = dev(want["lse"].astype(np.float32)), dev(want["coef"].astype(np.float32))
    rows = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    count = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.spo_loss_active_rows(coef, rows, count, ws_bytes(B.WS_ACTIVE_ROWS, T=T))
    torch.cuda.synchronize()
    n_act = int(count[0].item())
    want_rows = np.nonzero(want["coef"].astype(np.float32) != 0)[0]
    assert n_act == len(want_rows) and 0 < n_act < 0.7 * T
    np.testing.assert_array_equal(rows[:n_act].cpu().numpy(), want_rows)
    dH = torch.full((T, d), float("nan"), dtype=torch.float32 if dh_f32 else torch.bfloat16, device="cuda")
    dW = torch.full((V, d), float("nan"), dtype=torch.float32, device="cuda")
    st = status_word()
    B.spo_loss_bwd_rows(H, W, y, lse, coef, 0.7, rows, n_act, dH, dW, 0, ws_bytes(B.WS_LOSS_BWD_ROWS, T=n_act, d=d, V=V),
                        p, st)
    torch.cuda.synchronize()
    assert int(st[0].item()) == 0
    got_dh = dH.float().cpu().numpy()
    inactive = np.setdiff1d(np.arange(T), want_rows)
    assert np.all(got_dh[inactive] == 0.0)
    assert rel_fro(got_dh, want["dH"]) <= 1e-2
    assert rel_fro(dW.cpu().numpy(), want["dW"]) <= 1e-2


def test_row_lists_with_an_index_outside_the_batch_are_reported_not_dereferenced():
    """spo_loss_bwd_rows / spo_loss_fwd_bwd_rows take the row list from the caller: an entry outside
    [0, T) (a stale list, a list of another batch) sets the status bit and is skipped."""
    import torch
    from paper_2509_13232_b200 import binding as B
    from tests.helpers import dev, status_word, ws_bytes
    lb = _clip_batch(42, [60, 68], 64, 300, True)
    T, d, V, S = 128, 64, 300, 2
    H, W = dev(lb.h, torch.bfloat16), dev(lb.w, torch.bfloat16)
    y, lo, cu, an = dev(lb.y), dev(lb.logp_old), dev(lb.cu_seqlens), dev(lb.a_norm)
    f32 = dict(dtype=torch.float32, device="cuda")
    rows_host = np.arange(0, T, 2, dtype=np.int32)
    p = B.default_params()
    for bad in (-1, T, 2 ** 31 - 1):
        rows_bad = rows_host.copy()
        rows_bad[5] = bad
        rows = dev(rows_bad)
        n = len(rows_bad)
        loss = torch.zeros(4, **f32)
        logp, lse, coef = (torch.zeros(T, **f32) for _ in range(3))
        dH = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dW = torch.zeros((V, d), **f32)
        st = status_word()
        B.spo_loss_fwd_bwd_rows(H, W, y, lo, cu, an, rows, n, 1.0, loss, logp, lse, coef, None, dH, dW, 0,
                                ws_bytes(B.WS_LOSS_FWD_BWD_ROWS, T=n, d=d, V=V, B=S), p, st)
        torch.cuda.synchronize()
        assert int(st[0].item()) & B.DEV_ID_OUT_OF_RANGE
        assert torch.isfinite(dW).all() and torch.isfinite(dH.float()).all()
        st = status_word()
        B.spo_loss_bwd_rows(H, W, y, lse, coef, 1.0, rows, n, dH, dW, 0,
                            ws_bytes(B.WS_LOSS_BWD_ROWS, T=n, d=d, V=V), p, st)
        torch.cuda.synchronize()
        assert int(st[0].item()) & B.DEV_ID_OUT_OF_RANGE
        assert torch.isfinite(dW).all() and torch.isfinite(dH.float()).all()


def test_backward_over_active_rows_with_nothing_active():
    import torch
    from paper_2509_13232_b200 import binding as B
    from tests.helpers import dev, status_word, ws_bytes
    T, d, V = 300, 64, 200
    H = torch.randn((T, d), device="cuda").to(torch.bfloat16)
    W = torch.randn((V, d), device="cuda").to(torch.bfloat16)
    zeros = torch.zeros(T, device="cuda")
    rows = torch.zeros(T, dtype=torch.int32, device="cuda")
    count = torch.full((4,), 9, dtype=torch.int32, device="cuda")
    B.spo_loss_active_rows(zeros, rows, count, ws_bytes(B.WS_ACTIVE_ROWS, T=T))
    torch.cuda.synchronize()
    assert int(count[0].item()) == 0
    dH = torch.full((T, d), 1.0, dtype=torch.bfloat16, device="cuda")
    dW = torch.full((V, d), 1.0, device="cuda")
    B.spo_loss_bwd_rows(H, W, torch.zeros(T, dtype=torch.int32, device="cuda"), zeros, zeros, 1.0, rows, 0, dH, dW, 0,
                        ws_bytes(B.WS_LOSS_BWD_ROWS, T=0, d=d, V=V), B.default_params(), status_word())
    torch.cuda.synchronize()
    assert float(dH.float().abs().max().item()) == 0.0 and float(dW.abs().max().item()) == 0.0


def test_loss_stats_against_the_oracle():
    """Diagnostics of the update (mean ratio, clipped share, KL estimates, extreme ratios) from the forward's logp."""
    import torch
    from paper_2509_13232_b200 import binding as B
    from tests.helpers import dev
    lb = _clip_batch(170, [900, 1300, 0, 700, 2500, 61], 128, 1500, True)
    got = run_loss(lb)
    p = B.default_params()
    out = torch.full((8,), float("nan"), dtype=torch.float32, device="cuda")
    B.spo_loss_stats(dev(got["logp"]), dev(lb.logp_old), dev(lb.mask), dev(lb.cu_seqlens), dev(lb.a_norm), out, p)
    torch.cuda.synchronize()
    want = O.loss_stats(got["logp"], lb.logp_old, lb.mask, lb.cu_seqlens, lb.a_norm, float(np.float32(p.clip_lo)),
                        float(np.float32(p.clip_hi)))
    assert 0.02 < want[2] < 0.9 and want[7] >= want[2]
    np.testing.assert_allclose(out.cpu().numpy(), want, rtol=1e-5, atol=1e-6)
    # the share it reports as stopped is the share of unmasked tokens the forward gave a zero coef
    zero_adv = np.repeat(lb.a_norm, np.diff(lb.cu_seqlens)) == 0
    stopped = ((got["coef"] == 0) & (lb.mask != 0) & ~zero_adv).sum() / want[0]
    assert abs(stopped - want[2]) <= 2e-3              # tokens within rounding of a bound may fall on either side
    # nothing unmasked: zeros
    B.spo_loss_stats(dev(got["logp"]), dev(lb.logp_old), dev(np.zeros_like(lb.mask)), dev(lb.cu_seqlens), dev(lb.a_norm),
                     out, p)
    torch.cuda.synchronize()
    assert float(out.abs().max().item()) == 0.0
