"""Host-only checks of the C ABI: the library loads, exports what the header declares,
and rejects bad arguments before touching a device."""

import ctypes
import os
import re

import pytest

from paper_2509_13232_b200 import binding as B
from paper_2509_13232_b200 import build as spo_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    spo_build.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "spo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spo_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_default_params_are_the_papers(lib):
    p = B.default_params()
    assert abs(p.rho_min - 0.875) < 1e-7 and abs(p.rho_max - 0.96) < 1e-7
    assert abs(p.eps_explore - 0.05) < 1e-7
    assert abs(p.clip_lo - 0.2) < 1e-7 and abs(p.clip_hi - 0.28) < 1e-7
    assert p.norm_ddof == 0 and p.d_half > 0
    assert abs(p.near_zero_tau_lo - 1e-4) < 1e-10 and abs(p.near_zero_tau_hi - 0.02) < 1e-8   # Sec. 4 tolerances
    assert p.dual_clip == 0.0 and p.surrogate == B.SUR_PPO_CLIP and p.agg_mode == B.AGG_TOKEN_MEAN


def test_status_strings_and_version(lib):
    assert lib.spo_status_string(0) == b"ok"
    for code in range(-7, 0):
        assert lib.spo_status_string(code) not in (b"ok", b"unknown status")
    assert lib.spo_status_string(-99) == b"unknown status"
    assert lib.spo_version() >= 100


def test_workspace_sizes_are_monotone(lib):
    a = B.spo_workspace_bytes(B.WS_SAMPLE, N=1000, M=64)
    b = B.spo_workspace_bytes(B.WS_SAMPLE, N=1_000_000, M=8192)
    assert 0 < a < b
    assert B.spo_workspace_bytes(B.WS_ADVANTAGES, B=4096) > 0
    assert B.spo_workspace_bytes(B.WS_ADVANTAGES, B=1 << 20) >= B.spo_workspace_bytes(B.WS_ADVANTAGES, B=4096)
    f1 = B.spo_workspace_bytes(B.WS_LOSS_FWD, T=1000, d=128, V=5000)
    f2 = B.spo_workspace_bytes(B.WS_LOSS_FWD, T=100000, d=128, V=5000)
    assert 0 < f1 < f2
    # backward scratch is a bounded chunk: it stops growing with T
    g1 = B.spo_workspace_bytes(B.WS_LOSS_BWD, T=100_000, d=4096, V=151936)
    g2 = B.spo_workspace_bytes(B.WS_LOSS_BWD, T=1_000_000, d=4096, V=151936)
    assert g1 == g2 and g1 < 100_000 * 151936
    assert B.spo_workspace_bytes(99) == 0


def test_null_and_bad_arguments_are_rejected_on_the_host(lib):
    p = B.default_params()
    ref = ctypes.byref(p)
    assert lib.spo_default_params(None) == B.ERR_INVALID_ARG
    assert lib.spo_tracker_init(None, None, 5, ref, None) == B.ERR_INVALID_ARG
    assert lib.spo_tracker_init(None, None, -1, ref, None) == B.ERR_INVALID_ARG
    assert lib.spo_sample_prompts(None, 10, None, 4, 2, None, None, None, 0, ref, None, None) == B.ERR_INVALID_ARG
    fake = ctypes.c_void_p(0x1000)       # aligned, never dereferenced on the host
    odd = ctypes.c_void_p(0x1004)
    assert lib.spo_sample_prompts(fake, 10, fake, 1, 2, fake, None, fake, 1 << 20, ref, None, None) == B.ERR_BAD_SHAPE
    assert lib.spo_sample_prompts(odd, 10, fake, 4, 2, fake, None, fake, 1 << 20, ref, None, None) == B.ERR_BAD_ALIGNMENT
    assert lib.spo_advantages(fake, 10, fake, fake, 0, None, fake, None, None, 0, ref, None, None) == B.ERR_BAD_SHAPE
    assert lib.spo_tracker_update(fake, 10, fake, fake, fake, 2, 4, ref, None, None) == B.ERR_INVALID_ARG
    bad = B.default_params(rho_min=0.99, rho_max=0.9)
    assert lib.spo_tracker_update(fake, 10, fake, fake, fake, 0, 4, ctypes.byref(bad), None, None) == B.ERR_INVALID_ARG
    # loss: dtype, shape and alignment checks come before any device work
    args_tail = (fake, fake, fake, fake, fake, None, fake, 1 << 30, ref, None, None)
    assert lib.spo_loss_fwd(fake, fake, 7, fake, fake, None, fake, fake, 8, 64, 100, 1, *args_tail) == B.ERR_UNSUPPORTED_DTYPE
    assert lib.spo_loss_fwd(fake, fake, B.DTYPE_BF16, fake, fake, None, fake, fake, 8, 72, 100, 1, *args_tail) == B.ERR_BAD_SHAPE
    assert lib.spo_loss_fwd(odd, fake, B.DTYPE_BF16, fake, fake, None, fake, fake, 8, 64, 100, 1, *args_tail) == B.ERR_BAD_ALIGNMENT
    assert lib.spo_loss_bwd(fake, fake, B.DTYPE_BF16, fake, fake, fake, 1.0, 8, 64, 100, fake, 5, fake, 0,
                            fake, 1 << 30, ref, None, None) == B.ERR_UNSUPPORTED_DTYPE


def test_new_entry_points_reject_bad_arguments_on_the_host(lib):
    p = B.default_params()
    ref = ctypes.byref(p)
    fake = ctypes.c_void_p(0x1000)
    odd = ctypes.c_void_p(0x1004)
    # fused advantage + update
    assert lib.spo_advantages_update(None, 10, fake, fake, fake, 0, 4, None, fake, None, None, 0, ref, None, None) == B.ERR_INVALID_ARG
    assert lib.spo_advantages_update(fake, 10, fake, fake, fake, 3, 4, None, fake, None, None, 0, ref, None, None) == B.ERR_INVALID_ARG
    assert lib.spo_advantages_update(fake, 10, fake, fake, fake, 0, 0, None, fake, None, None, 0, ref, None, None) == B.ERR_BAD_SHAPE
    assert lib.spo_advantages_update(fake, 10, fake, odd, fake, 0, 4, None, fake, None, None, 0, ref, None, None) == B.ERR_BAD_ALIGNMENT
    # slab variant of the one-pass loss: the slab request is checked before anything else
    loss_args = (fake, fake, B.DTYPE_BF16, fake, fake, None, fake, fake, 8, 64, 100, 1, 1.0, fake, fake, fake, fake, None,
                 None, fake, B.DTYPE_BF16, fake, 0, fake, 1 << 40, ref, None, None)
    evs = (ctypes.c_void_p * 4)(fake, fake, fake, fake)
    assert lib.spo_loss_fwd_bwd_slabs(*loss_args, 0, evs) == B.ERR_INVALID_ARG
    assert lib.spo_loss_fwd_bwd_slabs(*loss_args, 65, evs) == B.ERR_INVALID_ARG
    assert lib.spo_loss_fwd_bwd_slabs(*loss_args, 4, None) == B.ERR_INVALID_ARG
    none_first = (ctypes.c_void_p * 4)(None, fake, fake, fake)
    assert lib.spo_loss_fwd_bwd_slabs(*loss_args, 4, none_first) == B.ERR_INVALID_ARG
    # reduce-scatter variant: the shard table is checked first
    assert lib.spo_loss_fwd_bwd_scatter(*loss_args, None) == B.ERR_INVALID_ARG
    sh = B.SpoDwShards()
    sh.n_shards, sh.rows_per_shard = 2, 10                       # 20 rows < V = 100
    sh.shard[0], sh.shard[1] = 0x1000, 0x2000
    assert lib.spo_loss_fwd_bwd_scatter(*loss_args, ctypes.byref(sh)) == B.ERR_INVALID_ARG
    sh.rows_per_shard = 50
    sh.shard[1] = None
    assert lib.spo_loss_fwd_bwd_scatter(*loss_args, ctypes.byref(sh)) == B.ERR_INVALID_ARG
    sh.shard[1] = 0x2004
    assert lib.spo_loss_fwd_bwd_scatter(*loss_args, ctypes.byref(sh)) == B.ERR_BAD_ALIGNMENT
    sh.n_shards = 17
    assert lib.spo_loss_fwd_bwd_scatter(*loss_args, ctypes.byref(sh)) == B.ERR_INVALID_ARG
    # parameters outside their domain
    for bad in (dict(dual_clip=1.0), dict(dual_clip=-2.0), dict(near_zero_tau_lo=-1.0), dict(surrogate=7)):
        q = B.default_params(**bad)
        assert lib.spo_advantages(fake, 10, fake, fake, 4, None, fake, None, None, 0, ctypes.byref(q), None, None) == B.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()
