"""GPU parity of the one-pass loss (spo_loss_fwd_bwd) against the CPU oracle.

Same oracle, same inputs and same tolerances as the two-call path (bf16: loss / logp / lse within
2e-3 absolute, gradients within 1e-2 relative Frobenius error; fp32: 1e-4 / 1e-4).  The one-pass
path stores the logits of a chunk as bf16 exponentials relative to one reference exponent per
row, so three things are checked beyond plain parity: the gradients keep their accuracy when
the logits span a wide range (a peaked, trained-model-like distribution), everything the
forward reports is independent of that storage (it agrees with the two-call forward to fp32
rounding), and a row whose logits outrun its reference is reported and skipped.
"""

import numpy as np
import pytest

from oracle import spo_oracle as O
from paper_2509_13232_b200 import inputs
from tests.helpers import oracle_loss, rel_fro, run_loss, worst_row_tile_error
from tests.test_gpu_loss import BF16_CASES, _clip_batch, check

pytestmark = pytest.mark.gpu


def test_cfg1_tiny_fp32_full_parity():
    tb, lb = inputs.cfg1_tiny()
    a0, b0 = O.tracker_init(tb.v0, 0.875)
    a_norm, _, _ = O.normalise_advantages(O.raw_advantage(a0, b0, tb.ids, tb.rewards))
    lb.a_norm = a_norm.astype(np.float32)
    check(lb, run_loss(lb, one_pass=True), oracle_loss(lb), 1e-4, 1e-4)


@pytest.mark.parametrize("name,lengths,d,v", BF16_CASES, ids=[c[0] for c in BF16_CASES])
def test_bf16_parity_small_shapes(name, lengths, d, v):
    lb = _clip_batch(20 + len(lengths) + d, lengths, d, v, True, w_std=0.05)
    got = run_loss(lb, grad_loss=0.6, one_pass=True)
    want = oracle_loss(lb, grad_loss=0.6)
    assert 0.02 < 1.0 - want["unclipped"].mean()
    check(lb, got, want, 2e-3, 1e-2)
    masked = lb.mask == 0
    assert masked.any() and np.all(got["dH"][masked] == 0.0)


def test_bf16_several_chunks_fp32_dh_and_dw_accumulate():
    """More token rows than one chunk holds, a ragged last chunk, dW added to what the buffer held."""
    lengths = [5000, 4100, 3000, 2900, 3100, 2207]
    lb = inputs.loss_batch(131, lengths, 128, 1200, 0.05, True, 0.3, target="softmax", mask_p=0.1)
    init = np.full((1200, 128), 0.25, dtype=np.float32)
    got = run_loss(lb, dh_bf16=False, dw_init=init, one_pass=True)
    want = oracle_loss(lb)
    assert got["status"] == 0 and lb.h.shape[0] > 2 * 9472
    assert abs(got["loss"] - want["loss"]) <= 2e-3
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)
    np.testing.assert_allclose(got["lse"], want["lse"], rtol=0, atol=2e-3)
    assert rel_fro(got["coef"], want["coef"]) <= 1e-2
    assert rel_fro(got["dH"], want["dH"]) <= 1e-2
    assert rel_fro(got["dW"] - init, want["dW"]) <= 1e-2
    scale = np.maximum(1.0, want["seq_sums"][:, 2:3])
    np.testing.assert_allclose(got["seq_sums"] / scale, want["seq_sums"] / scale, rtol=0, atol=2e-3)


def test_bf16_five_chunks_dw_contracted_two_chunks_at_a_time():
    """dW is contracted over two chunks of token rows per launch: five chunks give a storing launch over
    chunks 0 + 1, an adding one over 2 + 3 and an adding one over the short last chunk alone.  Checked
    against the oracle per 256-row vocabulary tile (the ragged last tile included), both with a fresh dW
    and on top of what the buffer held."""
    lengths = [9000, 7000, 5200, 8100, 6400, 4300, 2500, 1100]
    lb = inputs.loss_batch(137, lengths, 128, 1500, 0.05, True, 0.3, target="softmax", mask_p=0.1)
    assert 4 * 9472 < lb.h.shape[0] < 5 * 9472
    want = oracle_loss(lb)
    for init in (None, np.full((1500, 128), -0.5, dtype=np.float32)):
        got = run_loss(lb, dw_init=init, one_pass=True)
        assert got["status"] == 0
        assert abs(got["loss"] - want["loss"]) <= 2e-3
        np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)
        assert rel_fro(got["dH"], want["dH"]) <= 1e-2
        dw = got["dW"] if init is None else got["dW"] - init
        assert rel_fro(dw, want["dW"]) <= 1e-2
        worst, checked, n_tiles, last_checked = worst_row_tile_error(dw, want["dW"], 256)
        assert n_tiles == 6 and checked == 6 and last_checked and worst <= 2e-2


def test_forward_outputs_agree_with_the_two_call_path():
    """loss, logp, lse, coef come from fp32 accumulators in both paths; only the gradients see the
    stored exponentials."""
    lb = inputs.loss_batch(132, [3000, 700, 6100, 1500], 192, 5000, 0.05, True, 0.3, target="softmax", mask_p=0.2)
    a = run_loss(lb, grad_loss=1.3)
    b = run_loss(lb, grad_loss=1.3, one_pass=True)
    assert abs(a["loss"] - b["loss"]) <= 1e-6
    for k in ("logp", "lse"):
        np.testing.assert_allclose(a[k], b[k], rtol=0, atol=2e-5)
    np.testing.assert_allclose(a["coef"], b["coef"], rtol=1e-4, atol=1e-9)
    assert rel_fro(b["dH"], a["dH"]) <= 1e-2 and rel_fro(b["dW"], a["dW"]) <= 1e-2


@pytest.mark.parametrize("w_std", [0.5, 2.0])
def test_wide_logit_range_keeps_gradient_accuracy(w_std):
    """Logits spanning tens to hundreds of nats (peaked rows, as a trained model gives): the stored
    exponentials are taken against one reference per row and bf16 keeps its relative precision at
    any magnitude, so the probabilities that carry the gradient keep bf16 relative accuracy."""
    lb = inputs.loss_batch(133, [260, 300], 64, 3000, w_std, True, 0.1, target="softmax")
    z = lb.h.astype(np.float64) @ lb.w.astype(np.float64).T
    assert np.ptp(z, axis=1).mean() > 20.0
    got = run_loss(lb, one_pass=True)
    want = oracle_loss(lb)
    assert got["status"] == 0
    # absolute error of an fp32-accumulated logit grows with its size; allow 2e-3 per 16 nats
    tol = 2e-3 * max(1.0, np.abs(z).max() / 16.0)
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=tol)
    assert rel_fro(got["dH"], want["dH"]) <= 1e-2
    assert rel_fro(got["dW"], want["dW"]) <= 1e-2


def test_a_row_that_outruns_its_reference_exponent_is_reported_and_skipped():
    """The reference exponent of a row comes from its first 512 logits; a logit more than ~100 nats
    above them overflows the stored exponentials.  Such a row must set the status bit, get
    lse = Inf / logp = -Inf / coef = 0 and leave every gradient finite and, for all other rows,
    equal to the oracle's with that row's coefficient zeroed.  (The two-call path has no such limit.)"""
    from paper_2509_13232_b200 import binding as B
    lb = inputs.loss_batch(134, [150, 170], 64, 1500, 0.05, True, 0.1, target="softmax")
    t0, v0 = 77, 1000                                   # token row and a vocabulary row beyond the first tile
    u = np.zeros(64, dtype=np.float32)
    u[3] = 12.0
    lb.h[t0], lb.w[v0] = u, u                           # logit 144 there; the other rows see at most |12 h_3| < 60
    got = run_loss(lb, one_pass=True)
    assert got["status"] == B.DEV_NONFINITE
    assert np.isposinf(got["lse"][t0]) and np.isneginf(got["logp"][t0]) and got["coef"][t0] == 0.0
    assert np.all(got["dH"][t0] == 0.0) and np.all(np.isfinite(got["dH"])) and np.all(np.isfinite(got["dW"]))
    fwd = O.loss_forward(lb.h, lb.w, lb.y, lb.logp_old, lb.mask, lb.cu_seqlens, lb.a_norm)
    keep = np.arange(lb.h.shape[0]) != t0
    np.testing.assert_allclose(got["logp"][keep], fwd["logp"][keep], rtol=0, atol=4e-3)
    coef = fwd["coef"].copy()
    coef[t0] = 0.0
    dh, dw = O.loss_backward(lb.h, lb.w, lb.y, fwd["lse"], coef)
    assert rel_fro(got["coef"], coef) <= 1e-2
    assert rel_fro(got["dH"], dh) <= 1e-2 and rel_fro(got["dW"], dw) <= 1e-2
    # the two calls handle the same batch without a flag
    two = run_loss(lb, one_pass=False)
    assert two["status"] == 0 and abs(two["logp"][t0] - fwd["logp"][t0]) <= 2e-2


def test_bf16_uniform_logits_and_bad_target():
    lb = inputs.loss_batch(32, [50, 78], 64, 300, 0.05, True, 0.05, target="uniform")
    lb.w[:] = 0.0
    got = run_loss(lb, one_pass=True)
    np.testing.assert_allclose(got["logp"], -np.log(300.0), atol=1e-5)
    # W = 0: dH = coef (W_y - sum_v p W_v) = 0
    assert np.all(got["dH"] == 0.0)
    lb.y[3] = 300
    got = run_loss(lb, one_pass=True)
    assert got["status"] & 1
    assert np.isneginf(got["logp"][3]) and got["coef"][3] == 0.0 and np.all(got["dH"][3] == 0.0)


def test_empty_batch_is_a_no_op_with_zero_loss():
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
        dW = torch.full((v, d), 3.0, device="cuda")
        dH = torch.empty((0, d), dtype=dt, device="cuda")
        B.spo_loss_fwd_bwd(H, W, z(0, torch.int32), z(0), None, cu, z(0), 1.0, loss, z(0), z(0), z(0), None, dH, dW, 0,
                           ws_bytes(B.WS_LOSS_FWD_BWD, T=0, d=d, V=v, B=1), p, st)
        torch.cuda.synchronize()
        assert loss[0].item() == 0.0 and int(st[0].item()) == 0
        if dt == torch.bfloat16:
            assert float(dW.abs().max().item()) == 0.0


def test_all_tokens_masked_gives_zero_loss_and_zero_gradients():
    lb = inputs.loss_batch(51, [20, 13], 64, 200, 0.05, True, 0.1)
    lb.mask[:] = 0
    got = run_loss(lb, one_pass=True)
    want = oracle_loss(lb)
    assert want["loss"] == 0.0 and got["loss"] == 0.0 and got["status"] == 0
    assert np.all(got["coef"] == 0.0) and np.all(got["dH"] == 0.0) and np.all(got["dW"] == 0.0)
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)


def test_single_token_and_empty_sequences():
    one = inputs.loss_batch(52, [1], 64, 130, 0.05, True, 0.1)
    check(one, run_loss(one, one_pass=True), oracle_loss(one), 2e-3, 1e-2)
    gaps = inputs.loss_batch(53, [5, 0, 0, 9, 0, 3], 64, 130, 0.05, True, 0.3,
                             a_norm=np.array([1.0, 9.0, -9.0, -0.7, 5.0, 0.4], dtype=np.float32))
    got, want = run_loss(gaps, one_pass=True), oracle_loss(gaps)
    check(gaps, got, want, 2e-3, 1e-2)
    np.testing.assert_array_equal(got["seq_sums"][[1, 2, 4]], 0.0)


@pytest.mark.parametrize("v", [40, 64, 100, 512, 1024, 1025])
def test_bf16_vocabulary_edges(v):
    """Vocabulary below one 64-column group, exactly one, below one tile, one and two tiles, one over."""
    lb = _clip_batch(60 + v, [70, 61], 64, v, True)
    check(lb, run_loss(lb, one_pass=True), oracle_loss(lb), 2e-3, 1e-2)


def test_bf16_targets_on_group_half_and_tile_boundaries():
    lb = inputs.loss_batch(70, [64], 64, 1200, 0.05, True, 0.05, target="uniform")
    edges = [0, 7, 8, 31, 32, 63, 64, 255, 256, 511, 512, 767, 768, 1023, 1024, 1199]
    lb.y[:len(edges)] = edges
    z = lb.h.astype(np.float64) @ lb.w.astype(np.float64).T
    from scipy.special import log_softmax
    lb.logp_old[:] = log_softmax(z, axis=1)[np.arange(64), lb.y].astype(np.float32)
    got, want = run_loss(lb, one_pass=True), oracle_loss(lb)
    check(lb, got, want, 2e-3, 1e-2)
    np.testing.assert_allclose(want["ratio"], 1.0, atol=1e-6)


def test_sequence_mean_aggregation():
    from paper_2509_13232_b200 import binding as B
    params = B.default_params(agg_mode=B.AGG_SEQ_MEAN)
    lb = _clip_batch(90, [3, 40, 0, 17, 1, 9], 64, 333, True)
    lb.mask[3:43] = 0
    lb.mask[50] = 0
    got = run_loss(lb, params=params, grad_loss=0.8, one_pass=True)
    want = oracle_loss(lb, params=params, grad_loss=0.8)
    check(lb, got, want, 2e-3, 1e-2)
    got = run_loss(lb, params=params, mask_none=True, one_pass=True)
    want = oracle_loss(lb, params=params, mask_none=True)
    check(lb, got, want, 2e-3, 1e-2)


def test_results_are_bitwise_reproducible():
    lb = inputs.loss_batch(95, [2000, 1500, 1100, 97, 5300], 128, 1200, 0.05, True, 0.3, target="softmax", mask_p=0.1)
    a = run_loss(lb, grad_loss=0.9, one_pass=True)
    b = run_loss(lb, grad_loss=0.9, one_pass=True)
    assert a["loss"] == b["loss"]
    for k in ("logp", "lse", "coef", "dH", "dW", "seq_sums"):
        np.testing.assert_array_equal(a[k], b[k])


def test_results_do_not_depend_on_another_streams_kernels():
    """The CTA pairs of a launch pace one another, and their holds are bounded and advisory: when another
    stream's kernels take SMs away in the meantime (as a collective on a second stream would), the call
    still ends, reports nothing, and gives bit for bit what it gives alone."""
    import torch
    lengths = [5000, 4100, 3000, 2900, 3100, 2907]
    lb = inputs.loss_batch(96, lengths, 256, 4000, 0.05, True, 0.3, target="softmax", mask_p=0.1)
    alone = run_loss(lb, one_pass=True)
    assert alone["status"] == 0
    side = torch.cuda.Stream()
    x = torch.ones(32 << 20, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for _ in range(400):
            x.mul_(1.0001)
    busy = run_loss(lb, one_pass=True)          # on the current stream, while the other one is busy
    torch.cuda.synchronize()
    assert busy["status"] == 0 and busy["loss"] == alone["loss"]
    for k in ("logp", "lse", "coef", "dH", "dW"):
        np.testing.assert_array_equal(busy[k], alone[k])


def test_real_vocab_and_hidden_small_token_count_full_oracle():
    lb = inputs.loss_batch(41, [170, 1, 129], 4096, 151936, 0.02, True, 0.3, target="softmax", mask_p=0.1)
    got = run_loss(lb, one_pass=True)
    want = oracle_loss(lb)
    assert got["status"] == 0
    assert abs(got["loss"] - want["loss"]) <= 2e-3
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)
    np.testing.assert_allclose(got["lse"], want["lse"], rtol=0, atol=2e-3)
    assert rel_fro(got["coef"], want["coef"]) <= 1e-2
    assert rel_fro(got["dH"], want["dH"]) <= 1e-2
    assert rel_fro(got["dW"], want["dW"]) <= 1e-2
    assert np.abs(want["dW"][-64:]).max() > 0
    assert rel_fro(got["dW"][-64:], want["dW"][-64:]) <= 1e-2


def _run_rows(lb, params, grad_loss, dh_f32):
    """spo_loss_mask_rows + spo_loss_fwd_bwd_rows through the binding; numpy outputs."""
    import torch
    from paper_2509_13232_b200 import binding as B
    from tests.helpers import dev, status_word, ws_bytes
    H, W = dev(lb.h, torch.bfloat16), dev(lb.w, torch.bfloat16)
    T, d = H.shape
    V = W.shape[0]
    S = len(lb.cu_seqlens) - 1
    rows = torch.full((max(T, 1),), -1, dtype=torch.int32, device="cuda")
    count = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.spo_loss_mask_rows(dev(lb.mask), rows, count, ws_bytes(B.WS_ACTIVE_ROWS, T=T))
    torch.cuda.synchronize()
    n = int(count[0].item())
    f32 = dict(dtype=torch.float32, device="cuda")
    loss = torch.zeros(4, **f32)
    logp, lse, coef = (torch.full((max(T, 1),), float("nan"), **f32) for _ in range(3))
    seq = torch.zeros((max(S, 1), 3), **f32)
    dH = torch.full((max(T, 1), d), float("nan"), dtype=torch.float32 if dh_f32 else torch.bfloat16, device="cuda")
    dW = torch.full((V, d), float("nan"), **f32)
    st = status_word()
    B.spo_loss_fwd_bwd_rows(H, W, dev(lb.y), dev(lb.logp_old), dev(lb.cu_seqlens), dev(lb.a_norm), rows, n, grad_loss,
                            loss, logp, lse, coef, seq, dH[:T], dW, 0,
                            ws_bytes(B.WS_LOSS_FWD_BWD_ROWS, T=n, d=d, V=V, B=S), params, st)
    torch.cuda.synchronize()
    return {"rows": rows[:n].cpu().numpy(), "loss": float(loss[0].item()), "logp": logp[:T].cpu().numpy(),
            "lse": lse[:T].cpu().numpy(), "coef": coef[:T].cpu().numpy(), "seq_sums": seq[:S].cpu().numpy(),
            "dH": dH[:T].float().cpu().numpy(), "dW": dW.cpu().numpy(), "status": int(st[0].item())}


@pytest.mark.parametrize("agg,dh_f32", [(0, False), (1, True)])
def test_unmasked_rows_only_matches_the_masked_oracle(agg, dh_f32):
    """40 % of the tokens masked, one response masked entirely, an empty response, more listed rows
    than one chunk: the compacted one-pass call gives the oracle's loss, sums and gradients."""
    from paper_2509_13232_b200 import binding as B
    lb = _clip_batch(140, [5000, 1300, 0, 700, 9000, 61, 4100], 128, 1500, True)
    rng = np.random.default_rng(4)
    lb.mask[:] = (rng.random(lb.mask.shape[0]) > 0.4).astype(np.uint8)
    lb.mask[5000:6300] = 0
    params = B.default_params(agg_mode=agg)
    want = oracle_loss(lb, params=params, grad_loss=0.7)
    got = _run_rows(lb, params, 0.7, dh_f32)
    listed = np.nonzero(lb.mask)[0]
    np.testing.assert_array_equal(got["rows"], listed)
    assert got["status"] == 0 and len(listed) > 9472
    assert abs(got["loss"] - want["loss"]) <= 2e-3
    np.testing.assert_allclose(got["logp"][listed], want["logp"][listed], rtol=0, atol=2e-3)
    np.testing.assert_allclose(got["lse"][listed], want["lse"][listed], rtol=0, atol=2e-3)
    assert rel_fro(got["coef"], want["coef"]) <= 1e-2
    scale = np.maximum(1.0, want["seq_sums"][:, 2:3])
    np.testing.assert_allclose(got["seq_sums"] / scale, want["seq_sums"] / scale, rtol=0, atol=2e-3)
    hidden = np.setdiff1d(np.arange(lb.mask.shape[0]), listed)
    for k in ("logp", "lse", "coef"):
        assert np.all(got[k][hidden] == 0.0)
    assert np.all(got["dH"][hidden] == 0.0)
    assert rel_fro(got["dH"], want["dH"]) <= 1e-2
    assert rel_fro(got["dW"], want["dW"]) <= 1e-2


def test_unmasked_rows_only_with_everything_masked():
    from paper_2509_13232_b200 import binding as B
    lb = inputs.loss_batch(141, [20, 13], 64, 200, 0.05, True, 0.1)
    lb.mask[:] = 0
    got = _run_rows(lb, B.default_params(), 1.0, False)
    assert len(got["rows"]) == 0 and got["loss"] == 0.0 and got["status"] == 0
    for k in ("logp", "lse", "coef", "dH", "dW", "seq_sums"):
        assert np.all(got[k] == 0.0), k


@pytest.mark.parametrize("bf16,one_pass", [(True, True), (True, False), (False, False), (False, True)])
def test_policy_entropy_output(bf16, one_pass):
    """The optional per-token entropy of the softmax, accumulated in the contraction's epilogue:
    equal to the oracle's -sum p log p, on both loss paths and element types, over several chunks
    and a ragged vocabulary; asking for it changes no other output."""
    lengths = [5000, 4100, 897] if bf16 else [40, 25, 1]
    d, v = (128, 1211) if bf16 else (32, 257)
    lb = inputs.loss_batch(180, lengths, d, v, 0.3, bf16, 0.1, target="softmax", mask_p=0.1)
    want = oracle_loss(lb)
    assert want["entropy"].min() < 0.5 * np.log(v) and want["entropy"].max() > 0.5      # a spread of peaked and flat rows
    got = run_loss(lb, one_pass=one_pass, want_entropy=True)
    tol = 2e-3 if bf16 else 1e-4
    np.testing.assert_allclose(got["entropy"], want["entropy"], rtol=0, atol=tol)
    plain = run_loss(lb, one_pass=one_pass)
    assert plain["entropy"] is None and plain["loss"] == got["loss"]
    for k in ("logp", "lse", "coef"):
        np.testing.assert_array_equal(plain[k], got[k])
    assert rel_fro(got["dH"], plain["dH"]) <= 1e-6 and rel_fro(got["dW"], plain["dW"]) <= 1e-6


def test_policy_entropy_of_uniform_logits_is_log_v():
    lb = inputs.loss_batch(181, [50, 78], 64, 300, 0.05, True, 0.05, target="uniform")
    lb.w[:] = 0.0
    for one_pass in (False, True):
        got = run_loss(lb, one_pass=one_pass, want_entropy=True)
        np.testing.assert_allclose(got["entropy"], np.log(300.0), atol=1e-5)
