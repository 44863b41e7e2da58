"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The float64 oracle cannot run 244k tokens x 151936 vocabulary entries, so:
  * per-token outputs (logp, lse, coef, dH rows) are row-local: the oracle computes them one by
    one for sampled token rows (tile corners, chunk boundaries, random rows);
  * dW, which sums over all tokens, is checked (a) in full against the oracle at a shrunken
    token count with the real d and V, and (b) at full size through identities that hold at
    any size: the logit gradient of every token sums to zero over the vocabulary, so the
    columns of dW sum to zero, and <dW, W> = <dH, H> (both equal sum_t sum_v g[t,v] z[t,v]).
Tolerances: 2e-3 absolute on logp / lse / loss, 1e-2 relative Frobenius on gradients.
"""

import numpy as np
import pytest

from oracle import spo_oracle as O
from paper_2509_13232_b200 import inputs
from tests.helpers import oracle_loss, rel_fro, run_loss

pytestmark = pytest.mark.gpu


def test_real_vocab_and_hidden_small_token_count_full_oracle():
    lb = inputs.loss_batch(41, [170, 1, 129], 4096, 151936, 0.02, True, 0.3, target="softmax", mask_p=0.1)
    got = run_loss(lb)
    want = oracle_loss(lb)
    assert got["status"] == 0
    assert abs(got["loss"] - want["loss"]) <= 2e-3
    np.testing.assert_allclose(got["logp"], want["logp"], rtol=0, atol=2e-3)
    np.testing.assert_allclose(got["lse"], want["lse"], rtol=0, atol=2e-3)
    assert rel_fro(got["coef"], want["coef"]) <= 1e-2
    assert rel_fro(got["dH"], want["dH"]) <= 1e-2
    assert rel_fro(got["dW"], want["dW"]) <= 1e-2
    # the ragged last vocabulary tile (V = 593.5 tiles of 256) carries gradient too
    assert np.abs(want["dW"][-64:]).max() > 0
    assert rel_fro(got["dW"][-64:], want["dW"][-64:]) <= 1e-2


@pytest.mark.parametrize("path", ["onepass", "split"])
@pytest.mark.parametrize("workload", ["cfg3_small_bf16", "cfg4_8b_bf16", "cfg5_longtail_bf16"])
def test_full_size_sampled_rows_and_identities(workload, path):
    """Both loss paths bench.py can time: one spo_loss_fwd_bwd call, or spo_loss_fwd then spo_loss_bwd."""
    import torch
    import bench
    step = bench.Step(workload, torch.device("cuda", 0), 0, path=path)
    step.run()
    torch.cuda.synchronize()
    assert int(step.status[0].item()) == 0
    D, T, S = step.data, step.T, step.S
    p = step.params
    # tracker pieces of the step from the oracle (table as it stood before the step)
    ab0 = step.ab0.cpu().numpy()
    w32 = O.sampling_weights_f32(ab0[:, 0], ab0[:, 1], np.float32(p.eps_explore))
    ids = O.sample_prompts(w32, step.uniforms.cpu().numpy(), S)
    np.testing.assert_array_equal(step.ids.cpu().numpy(), ids)
    rewards = step.rewards.cpu().numpy()
    raw = O.raw_advantage(ab0[:, 0].astype(np.float64), ab0[:, 1].astype(np.float64), ids, rewards)
    a_norm, _, _ = O.normalise_advantages(raw, 0, float(np.float32(p.norm_eps)))
    np.testing.assert_allclose(step.a_norm.cpu().numpy(), a_norm, rtol=1e-5, atol=2e-6)
    kl = step.kl_table.cpu().numpy()[ids].astype(np.float64)
    a1, b1 = O.tracker_update(ab0[:, 0].astype(np.float64), ab0[:, 1].astype(np.float64), ids, rewards, kl,
                              float(np.float32(p.d_half)))
    ab1 = step.ab.cpu().numpy()
    np.testing.assert_allclose(ab1[ids, 0], a1[ids], rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(ab1[ids, 1], b1[ids], rtol=1e-5, atol=1e-6)

    # sampled token rows: corners of token tiles, both sides of backward-chunk boundaries, random rows
    chunk = -(-T // step.bwd_chunks)
    chunk = (step.ws_bwd_bytes // (((step.V + 255) // 256) * 256 * 2))
    rng = np.random.default_rng(5)
    rows = sorted(set([0, 127, 128, chunk - 1, chunk, 2 * chunk - 1, T - 1, T - 2] +
                      rng.integers(0, T, 16).tolist()))
    rows_t = torch.tensor(rows, device="cuda")
    cu = D["cu_seqlens"].cpu().numpy()
    seq = O.token_sequence_ids(cu, T)[rows]
    w_host = D["w"].float().cpu().numpy()
    sub = O.loss_rows(D["h"][rows_t].float().cpu().numpy(), w_host, D["y"][rows_t].cpu().numpy(),
                      D["logp_old"][rows_t].cpu().numpy(), np.ones(len(rows)), a_norm[seq], float(step.n_tok))
    np.testing.assert_allclose(step.logp[rows_t].cpu().numpy(), sub["logp"], rtol=0, atol=2e-3)
    np.testing.assert_allclose(step.lse[rows_t].cpu().numpy(), sub["lse"], rtol=0, atol=2e-3)
    assert rel_fro(step.coef[rows_t].cpu().numpy(), sub["coef"]) <= 1e-2
    got_dh = step.dH[rows_t].float().cpu().numpy()
    for i in range(len(rows)):
        assert rel_fro(got_dh[i], sub["dH"][i]) <= 1e-2, rows[i]

    # loss: the fixed-order reduction against a float64 fold of the per-token terms
    logp = step.logp.double()
    ratio = torch.exp(logp - D["logp_old"].double())
    a_tok = torch.from_numpy(a_norm).cuda()[torch.from_numpy(O.token_sequence_ids(cu, T)).cuda()]
    sur = torch.minimum(ratio * a_tok, torch.clamp(ratio, 1 - 0.2, 1 + 0.28) * a_tok)
    assert abs(float(step.loss[0].item()) + float(sur.mean().item())) <= 2e-3

    # identities on dW at full size
    dW = step.dW
    col = dW.double().sum(dim=0)
    scale = dW.double().abs().sum(dim=0)
    assert float((col.abs() / scale.clamp_min(1e-30)).max().item()) <= 1e-2
    # <dW, W> = <dH, H>.  Both sums cancel heavily (sum_v g z is a small difference of large
    # terms), so the comparison is scaled by the un-cancelled magnitude sum |dW o W|.
    prod = dW.double() * D["w"].double()
    lhs, mag = float(prod.sum().item()), float(prod.abs().sum().item())
    del prod
    rhs = 0.0
    for t0 in range(0, T, 32768):
        rhs += float((step.dH[t0:t0 + 32768].double() * D["h"][t0:t0 + 32768].double()).sum().item())
    assert abs(lhs - rhs) <= 1e-3 * mag


@pytest.mark.parametrize("path", ["onepass", "split"])
def test_full_size_step_is_bitwise_reproducible(path):
    """Two runs of the whole step at the cfg3 workload (eight chunks, lock-stepped CTA pairs, side warps,
    chunk-by-chunk dW accumulation): every output identical bit for bit."""
    import torch
    import bench
    step = bench.Step("cfg3_small_bf16", torch.device("cuda", 0), 0, path=path)
    outs = []
    for _ in range(2):
        step.ab.copy_(step.ab0)
        step.run()
        torch.cuda.synchronize()
        outs.append([t.clone() for t in (step.loss, step.logp, step.lse, step.coef, step.dH, step.dW, step.ids, step.ab)])
    assert int(step.status[0].item()) == 0
    for a, b in zip(*outs):
        assert torch.equal(a, b)
