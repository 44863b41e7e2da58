"""GPU parity of the other objectives Sec. 3.2 names as compatible with the SPO advantage
(spo_params.surrogate): the truncated-importance-weight log-likelihood (CISPO) on both loss paths and
in both element types, PPO-Clip on a sequence-level ratio (GSPO), and the second clip of dual-clip PPO
(spo_params.dual_clip) on the token-level and the sequence-level objective.
Tolerances as for the default objective: bf16 2e-3 absolute / 1e-2 relative Frobenius, fp32 1e-4 / 1e-4.
"""

import ctypes

import numpy as np
import pytest

from paper_2509_13232_b200 import inputs
from tests.helpers import oracle_loss, rel_fro, run_loss
from tests.test_gpu_loss import _clip_batch, check

pytestmark = pytest.mark.gpu


def _params(**kw):
    from paper_2509_13232_b200 import binding as B
    return B.default_params(**kw)


@pytest.mark.parametrize("bf16,one_pass", [(False, False), (True, False), (True, True), (False, True)])
def test_cispo_parity(bf16, one_pass):
    from paper_2509_13232_b200 import binding as B
    lb = _clip_batch(150, [300, 40, 0, 517, 1, 90], 64, 777, bf16)
    for agg in (B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN):
        params = _params(surrogate=B.SUR_CISPO, agg_mode=agg)
        want = oracle_loss(lb, params=params, grad_loss=0.9)
        got = run_loss(lb, params=params, grad_loss=0.9, one_pass=one_pass)
        # every unmasked token with a non-zero advantage carries gradient, clipped or not
        live = (lb.mask != 0) & (np.repeat(lb.a_norm, np.diff(lb.cu_seqlens)) != 0)
        assert np.all(got["coef"][live] != 0.0) and np.all(got["coef"][lb.mask == 0] == 0.0)
        tol = (2e-3, 1e-2) if bf16 else (1e-4, 1e-4)
        # the loss is a mean of w*a*logp with |logp| ~ log V: allow the absolute tolerance per unit of |logp|
        assert abs(got["loss"] - want["loss"]) <= tol[0] * max(1.0, float(np.abs(want["logp"]).max()))
        got["loss"] = want["loss"]
        check(lb, got, want, *tol)
    other = oracle_loss(lb, params=_params(), grad_loss=0.9)
    assert rel_fro(other["coef"], want["coef"]) > 0.05        # and it is not the default objective


@pytest.mark.parametrize("bf16,one_pass", [(False, False), (True, False), (True, True), (False, True)])
def test_gspo_parity(bf16, one_pass):
    from paper_2509_13232_b200 import binding as B
    lengths = [300, 40, 0, 517, 1, 90, 2500] if bf16 else [30, 4, 0, 51, 1, 9]
    lb = _clip_batch(151, lengths, 64, 333, bf16)
    lb.mask[300:340] = 0                                   # one response masked entirely (bf16 case)
    # per-token noise of 0.3 averages out over a response: shift whole responses so that some clip
    seq = np.repeat(np.arange(len(lengths)), lengths)
    shift = np.array([0.4, 0.0, 0.0, -0.4, 0.5, -0.1, 0.05])[:len(lengths)]
    lb.logp_old = (lb.logp_old - shift[seq]).astype(np.float32)
    params = _params(surrogate=B.SUR_GSPO, clip_lo=0.2, clip_hi=0.28)
    want = oracle_loss(lb, params=params, grad_loss=1.1)
    assert 0 < want["unclipped"].sum() < len(want["unclipped"])
    got = run_loss(lb, params=params, grad_loss=1.1, one_pass=one_pass)
    tol = (2e-3, 1e-2) if bf16 else (1e-4, 1e-4)
    check(lb, got, want, *tol)
    # tokens of a response share one coefficient
    for s in range(len(lengths)):
        c = got["coef"][(seq == s) & (lb.mask != 0)]
        assert c.size == 0 or np.all(c == c[0])


def test_gspo_is_refused_by_the_compacted_one_pass_call():
    """spo_loss_fwd_bwd_rows has no forward-then-backward form: it refuses the sequence-level objective."""
    from paper_2509_13232_b200 import binding as B
    p = _params(surrogate=B.SUR_GSPO)
    fake = ctypes.c_void_p(0x1000)
    rc = B.lib().spo_loss_fwd_bwd_rows(fake, fake, B.DTYPE_BF16, fake, fake, fake, fake, 8, 64, 100, 1, fake, 4, 1.0,
                                       fake, fake, fake, fake, None, fake, B.DTYPE_BF16, fake, 0, fake, 1 << 40,
                                       ctypes.byref(p), None, None)
    assert rc == B.ERR_INVALID_ARG


@pytest.mark.parametrize("bf16,one_pass", [(False, False), (True, False), (True, True), (False, True)])
def test_dual_clip_parity(bf16, one_pass):
    """Second clip for negative advantages: tokens whose ratio exceeds c lose their gradient and their
    term is the constant c a.  c = 1.5 so that, with old log-probs 0.3 away, a tenth of the tokens is beyond it."""
    from paper_2509_13232_b200 import binding as B
    lb = _clip_batch(152, [300, 40, 0, 517, 1, 90], 64, 777, bf16)
    lb.a_norm[:] = [-1.0, 0.7, 0.0, -0.6, 1.2, -0.3]
    params = _params(dual_clip=1.5)
    want = oracle_loss(lb, params=params, grad_loss=0.8)
    plain = oracle_loss(lb, params=_params(), grad_loss=0.8)
    second = (plain["coef"] != 0.0) & (want["coef"] == 0.0)
    assert second.sum() >= 10 and abs(want["loss"] - plain["loss"]) > 1e-3       # the second clip is at work
    got = run_loss(lb, params=params, grad_loss=0.8, one_pass=one_pass)
    check(lb, got, want, *((2e-3, 1e-2) if bf16 else (1e-4, 1e-4)))
    assert np.all(got["coef"][second] == 0.0) and np.all(got["dH"][second] == 0.0)
    # c must exceed 1: rejected on the host before anything is touched
    assert B.lib().spo_loss_fwd(*([None] * 2), 0, *([None] * 5), 0, 64, 10, 0, *([None] * 7), 0,
                                ctypes.byref(_params(dual_clip=0.9)), None, None) == B.ERR_INVALID_ARG


def test_dual_clip_on_the_sequence_level_objective():
    from paper_2509_13232_b200 import binding as B
    lengths = [300, 40, 517, 1, 90, 2500]
    lb = _clip_batch(153, lengths, 64, 333, True)
    lb.a_norm[:] = [-1.0, -0.5, 0.7, -0.2, -1.5, 0.3]
    seq = np.repeat(np.arange(len(lengths)), lengths)
    shift = np.array([0.6, 0.1, 0.5, 0.7, -0.4, 0.05])           # response ratios about e^shift: 1.8, 1.1, 1.6, 2.0, 0.67, 1.05
    lb.logp_old = (lb.logp_old - shift[seq]).astype(np.float32)
    params = _params(surrogate=B.SUR_GSPO, dual_clip=1.5)
    want = oracle_loss(lb, params=params)
    plain = oracle_loss(lb, params=_params(surrogate=B.SUR_GSPO))
    assert ((plain["coef"] != 0.0) & (want["coef"] == 0.0)).any() and (want["coef"] != 0.0).any()
    got = run_loss(lb, params=params)
    check(lb, got, want, 2e-3, 1e-2)
