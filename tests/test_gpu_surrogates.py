"""GPU parity of the other objectives Sec. 3.2 names as compatible with the SPO advantage
(spo_params.surrogate): the truncated-importance-weight log-likelihood (CISPO) on both loss paths and
in both element types, and PPO-Clip on a sequence-level ratio (GSPO) on the two-call path.
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


@pytest.mark.parametrize("bf16", [False, True])
def test_gspo_parity_two_call_path(bf16):
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
    got = run_loss(lb, params=params, grad_loss=1.1)
    tol = (2e-3, 1e-2) if bf16 else (1e-4, 1e-4)
    check(lb, got, want, *tol)
    # tokens of a response share one coefficient
    for s in range(len(lengths)):
        c = got["coef"][(seq == s) & (lb.mask != 0)]
        assert c.size == 0 or np.all(c == c[0])


def test_gspo_is_refused_by_the_one_pass_call_for_bf16():
    import torch
    from paper_2509_13232_b200 import binding as B
    p = _params(surrogate=B.SUR_GSPO)
    fake = ctypes.c_void_p(0x1000)
    rc = B.lib().spo_loss_fwd_bwd(fake, fake, B.DTYPE_BF16, fake, fake, None, fake, fake, 8, 64, 100, 1, 1.0, fake, fake,
                                  fake, fake, None, None, fake, B.DTYPE_BF16, fake, 0, fake, 1 << 40, ctypes.byref(p), None, None)
    assert rc == B.ERR_INVALID_ARG
    assert torch.cuda.is_available()
