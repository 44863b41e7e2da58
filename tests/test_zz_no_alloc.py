"""spo_advantages_static -- the entry point for callers that cannot allocate device memory.

Some users of this library run where no scratch buffer can be produced: all free HBM already
belongs to a framework's caching allocator, or the call site is handed tensors but no
allocator.  For them the library keeps the partial sums of the advantage statistics in a
fixed device array of its own.  This test calls that entry point through the C ABI twice in
a row on different batches and requires the same results as spo_advantages (which takes
caller scratch) and as the CPU oracle (raw advantage with the pre-update baseline, then the
batch-global normalisation of Sec. 3.2), within the tolerances the other advantage tests
use.  The second call also shows that whatever the first call left in the shared array does
no harm.  Around the calls the driver's count of free device memory is read: it must not
move, since the whole point of the entry point is that it obtains no memory.  The file name
sorts last so that a run stopping at the first failure has already run everything else.
"""

import numpy as np
import pytest

from oracle import spo_oracle as O
from tests.helpers import dev, status_word, ws_bytes

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 2e-6


def _both(ab_t, ids, r, params, want_raw):
    import torch
    from paper_2509_13232_b200 import binding as B
    b = len(ids)
    f32 = dict(dtype=torch.float32, device="cuda")
    ids_t, r_t = dev(ids), dev(r)
    out = []
    for static in (False, True):
        a_raw = torch.full((b,), float("nan"), **f32) if want_raw else None
        a_norm = torch.full((b,), float("nan"), **f32)
        stats = torch.zeros(8, **f32)
        st = status_word()
        if static:
            B.spo_advantages_static(ab_t, ids_t, r_t, a_raw, a_norm, stats, params, st)
        else:
            B.spo_advantages(ab_t, ids_t, r_t, a_raw, a_norm, stats, ws_bytes(B.WS_ADVANTAGES, B=b), params, st)
        torch.cuda.synchronize()
        out.append((None if a_raw is None else a_raw.cpu().numpy(), a_norm.cpu().numpy(), stats.cpu().numpy(),
                    int(st[0].item())))
    return out


def test_static_scratch_entry_point_matches_the_allocating_one_twice():
    from paper_2509_13232_b200 import binding as B
    import torch
    rng = np.random.default_rng(2024)
    n = 400_000
    ab = rng.uniform(0.05, 14.0, (n, 2)).astype(np.float32)
    ab_t = dev(ab)
    a64, b64 = ab[:, 0].astype(np.float64), ab[:, 1].astype(np.float64)
    # two calls in a row: a large batch (many partial blocks), then a small one with other settings
    cases = [(250_000, 0, True, 0.4), (3_000, 1, False, 0.7)]
    for b, ddof, want_raw, p_reward in cases:
        ids = rng.permutation(n)[:b].astype(np.int32)
        r = (rng.random(b) < p_reward).astype(np.float32)
        params = B.default_params(norm_ddof=ddof)
        (raw0, norm0, stats0, st0), (raw1, norm1, stats1, st1) = _both(ab_t, ids, r, params, want_raw)
        assert st0 == 0 and st1 == 0
        if want_raw:
            np.testing.assert_allclose(raw1, raw0, rtol=RTOL, atol=ATOL)
        np.testing.assert_allclose(norm1, norm0, rtol=RTOL, atol=ATOL)
        np.testing.assert_allclose(stats1, stats0, rtol=RTOL, atol=ATOL)
        assert abs(float(norm1.mean())) < 1e-4
        # ... and the same as the oracle's definition
        want_raw_v = O.raw_advantage(a64, b64, ids, r)
        want_norm, mu, sigma = O.normalise_advantages(want_raw_v, ddof, float(np.float32(params.norm_eps)))
        if want_raw:
            np.testing.assert_allclose(raw1, want_raw_v, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(norm1, want_norm, rtol=1e-5, atol=2e-6)
        np.testing.assert_allclose(stats1[:3], [mu, sigma, b], rtol=1e-5, atol=1e-6)


def test_static_scratch_entry_point_takes_no_device_memory():
    """Free device memory as the driver counts it is the same before and after two calls (outputs
    allocated beforehand; the first call of the process, which looks up the array's address, is
    made before the reading so that loading the library's device code is not mistaken for an
    allocation)."""
    import torch
    from paper_2509_13232_b200 import binding as B
    rng = np.random.default_rng(7)
    n, b = 100_000, 60_000
    ab_t = dev(rng.uniform(0.05, 14.0, (n, 2)).astype(np.float32))
    ids_t = dev(rng.permutation(n)[:b].astype(np.int32))
    r_t = dev((rng.random(b) < 0.5).astype(np.float32))
    a_norm = torch.empty(b, dtype=torch.float32, device="cuda")
    stats = torch.zeros(8, dtype=torch.float32, device="cuda")
    st = status_word()
    params = B.default_params()
    B.spo_advantages_static(ab_t, ids_t, r_t, None, a_norm, stats, params, st)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(2):
        B.spo_advantages_static(ab_t, ids_t, r_t, None, a_norm, stats, params, st)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert int(st[0].item()) == 0


def test_static_scratch_entry_point_rejects_oversized_batches():
    import ctypes
    from paper_2509_13232_b200 import binding as B
    p = B.default_params()
    fake = ctypes.c_void_p(0x1000)        # never dereferenced: the size check comes first
    rc = B.lib().spo_advantages_static(fake, 10, fake, fake, B.ADVANTAGES_STATIC_MAX_B + 1, None, fake, None,
                                       ctypes.byref(p), None, None)
    assert rc == B.ERR_BAD_SHAPE
