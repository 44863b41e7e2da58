"""ctypes binding of libspo.so: one Python function per C entry point, same names.

Argument marshalling only.  Tensors are torch CUDA tensors used as device
buffers (``data_ptr()``), the stream is torch's current stream; every step of
the path runs inside the library's CUDA kernels.  There is no CPU fallback: if
the shared library has not been built, loading it raises.
"""

from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int32, c_int64, c_size_t, c_void_p

# SPO_LIBRARY_PATH points at another build of the same library (e.g. one compiled with different tile options).
_LIB_PATH = os.environ.get("SPO_LIBRARY_PATH") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libspo.so")

SPO_OK = 0
ERR_INVALID_ARG, ERR_BAD_SHAPE, ERR_BAD_ALIGNMENT = -1, -2, -3
ERR_UNSUPPORTED_DTYPE, ERR_UNSUPPORTED_ARCH, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA = -4, -5, -6, -7
DEV_ID_OUT_OF_RANGE, DEV_NONFINITE, DEV_UNIFORMS_EXHAUSTED, DEV_TIMEOUT, DEV_ZERO_TOTAL_WEIGHT = 1, 2, 4, 8, 16
DTYPE_F32, DTYPE_BF16 = 0, 1
(WS_SAMPLE, WS_ADVANTAGES, WS_LOSS_FWD, WS_LOSS_BWD, WS_UPDATE_REPEATS, WS_ACTIVE_ROWS, WS_LOSS_BWD_ROWS,
 WS_LOSS_FWD_BWD, WS_LOSS_FWD_BWD_ROWS) = range(9)
AGG_TOKEN_MEAN, AGG_SEQ_MEAN = 0, 1
SUR_PPO_CLIP, SUR_CISPO, SUR_GSPO = 0, 1, 2

EXPORTS = [
    "spo_default_params", "spo_tracker_init", "spo_sample_prompts", "spo_advantages",
    "spo_advantages_static", "spo_advantages_apply", "spo_advantages_update",
    "spo_tracker_update", "spo_tracker_update_repeats", "spo_loss_fwd", "spo_loss_bwd", "spo_loss_fwd_bwd", "spo_loss_fwd_bwd_slabs", "spo_dw_slab_rows", "spo_loss_fwd_bwd_scatter", "spo_loss_stats", "spo_loss_mask_rows", "spo_loss_fwd_bwd_rows", "spo_loss_active_rows", "spo_loss_bwd_rows", "spo_workspace_bytes",
    "spo_status_string", "spo_last_cuda_error", "spo_version", "spo_selftest_bounded_wait",
]


class SpoParams(Structure):
    _fields_ = [
        ("rho_min", c_float), ("rho_max", c_float), ("d_half", c_float), ("eps_explore", c_float),
        ("clip_lo", c_float), ("clip_hi", c_float), ("norm_eps", c_float), ("norm_ddof", c_int32),
        ("agg_mode", c_int32), ("global_tokens", c_int32), ("global_responses", c_int32),
        ("surrogate", c_int32), ("dual_clip", c_float), ("near_zero_tau_lo", c_float),
        ("near_zero_tau_hi", c_float),
    ]


MAX_DW_SHARDS = 16


class SpoDwShards(Structure):
    _fields_ = [("n_shards", c_int32), ("rows_per_shard", c_int64), ("shard", c_void_p * MAX_DW_SHARDS)]


class SpoError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().spo_status_string(status).decode()
        if status == ERR_CUDA:
            msg += " [cudaError %d]" % lib().spo_last_cuda_error()
        super().__init__("%s: %s (%d)" % (where, msg, status))


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                "libspo.so is missing (%s): build it with `python -m paper_2509_13232_b200.build`; "
                "there is no fallback path" % _LIB_PATH)
        L = ctypes.CDLL(_LIB_PATH)
        P = POINTER(SpoParams)
        L.spo_default_params.argtypes = [P]
        L.spo_tracker_init.argtypes = [c_void_p, c_void_p, c_int64, P, c_void_p]
        L.spo_sample_prompts.argtypes = [c_void_p, c_int64, c_void_p, c_int32, c_int32, c_void_p, c_void_p,
                                         c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_advantages.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_int32, c_void_p, c_void_p,
                                     c_void_p, c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_advantages_static.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_int32, c_void_p, c_void_p,
                                            c_void_p, P, c_void_p, c_void_p]
        L.spo_advantages_update.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                                            c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_advantages_apply.argtypes = [c_void_p, c_int32, c_float, c_float, c_void_p, P, c_void_p]
        L.spo_tracker_update.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                                         P, c_void_p, c_void_p]
        L.spo_tracker_update_repeats.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                                                 c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_loss_fwd.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                   c_int64, c_int32, c_int32, c_int32,
                                   c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                   c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_loss_bwd.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_float,
                                   c_int64, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_int32,
                                   c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_loss_fwd_bwd.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                       c_int64, c_int32, c_int32, c_int32, c_float,
                                       c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                       c_void_p, c_int32, c_void_p, c_int32,
                                       c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_loss_fwd_bwd_slabs.argtypes = list(L.spo_loss_fwd_bwd.argtypes) + [c_int32, POINTER(c_void_p)]
        L.spo_loss_fwd_bwd_scatter.argtypes = list(L.spo_loss_fwd_bwd.argtypes) + [POINTER(SpoDwShards)]
        L.spo_dw_slab_rows.argtypes = [c_int32, c_int32, c_int32, POINTER(c_int64)]
        L.spo_loss_stats.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int32, c_void_p, P,
                                     c_void_p]
        L.spo_loss_mask_rows.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.spo_loss_fwd_bwd_rows.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                            c_int64, c_int32, c_int32, c_int32, c_void_p, c_int64, c_float,
                                            c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                            c_void_p, c_int32, c_void_p, c_int32,
                                            c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_loss_active_rows.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.spo_loss_bwd_rows.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_float,
                                        c_int64, c_int32, c_int32, c_void_p, c_int64, c_void_p, c_int32, c_void_p,
                                        c_int32, c_void_p, c_size_t, P, c_void_p, c_void_p]
        L.spo_selftest_bounded_wait.argtypes = [ctypes.c_uint32, c_void_p, c_void_p, c_void_p]
        L.spo_workspace_bytes.argtypes = [c_int32, c_int64, c_int32, c_int32, c_int64, c_int32, c_int32]
        L.spo_workspace_bytes.restype = c_size_t
        L.spo_status_string.argtypes = [c_int32]
        L.spo_status_string.restype = c_char_p
        for name in EXPORTS:
            if name not in ("spo_workspace_bytes", "spo_status_string"):
                getattr(L, name).restype = c_int32
        _lib = L
    return _lib


def default_params(**overrides) -> SpoParams:
    p = SpoParams()
    rc = lib().spo_default_params(ctypes.byref(p))
    if rc != SPO_OK:
        raise SpoError(rc, "spo_default_params")
    for k, v in overrides.items():
        setattr(p, k, v)
    return p


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream():
    import torch
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, where):
    if rc != SPO_OK:
        raise SpoError(rc, where)


def _dtype_code(t):
    import torch
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float32:
        return DTYPE_F32
    raise TypeError("H/W/dH must be float32 or bfloat16, got %s" % t.dtype)


def spo_workspace_bytes(which, T=0, d=0, V=0, N=0, B=0, M=0) -> int:
    return int(lib().spo_workspace_bytes(which, T, d, V, N, B, M))


def spo_tracker_init(ab, v0, params):
    _check(lib().spo_tracker_init(_ptr(ab), _ptr(v0), v0.numel(), ctypes.byref(params), _stream()),
           "spo_tracker_init")


def spo_sample_prompts(ab, uniforms, B, out_ids, out_w, ws, params, d_status):
    _check(lib().spo_sample_prompts(_ptr(ab), ab.shape[0], _ptr(uniforms), uniforms.numel(), B, _ptr(out_ids),
                                    _ptr(out_w), _ptr(ws), ws.numel() * ws.element_size(), ctypes.byref(params),
                                    _ptr(d_status), _stream()), "spo_sample_prompts")


def spo_advantages(ab, ids, r, a_raw, a_norm, stats, ws, params, d_status):
    _check(lib().spo_advantages(_ptr(ab), ab.shape[0], _ptr(ids), _ptr(r), ids.numel(), _ptr(a_raw), _ptr(a_norm),
                                _ptr(stats), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                ctypes.byref(params), _ptr(d_status), _stream()), "spo_advantages")


def spo_advantages_update(ab, ids, r, kl, kl_is_table, a_raw, a_norm, stats, ws, params, d_status):
    _check(lib().spo_advantages_update(_ptr(ab), ab.shape[0], _ptr(ids), _ptr(r), _ptr(kl), int(kl_is_table),
                                       ids.numel(), _ptr(a_raw), _ptr(a_norm), _ptr(stats), _ptr(ws),
                                       0 if ws is None else ws.numel() * ws.element_size(), ctypes.byref(params),
                                       _ptr(d_status), _stream()), "spo_advantages_update")


def spo_advantages_apply(a_raw, mu, sigma, a_norm, params):
    _check(lib().spo_advantages_apply(_ptr(a_raw), a_raw.numel(), c_float(mu), c_float(sigma), _ptr(a_norm),
                                      ctypes.byref(params), _stream()), "spo_advantages_apply")


ADVANTAGES_STATIC_MAX_B = 4194304


def spo_advantages_static(ab, ids, r, a_raw, a_norm, stats, params, d_status):
    """spo_advantages for callers that cannot supply scratch memory: same inputs and outputs,
    no `ws`; the library's own fixed device array holds the partial sums (B <= ADVANTAGES_STATIC_MAX_B;
    calls must not overlap on the GPU)."""
    _check(lib().spo_advantages_static(_ptr(ab), ab.shape[0], _ptr(ids), _ptr(r), ids.numel(), _ptr(a_raw),
                                       _ptr(a_norm), _ptr(stats), ctypes.byref(params), _ptr(d_status),
                                       _stream()), "spo_advantages_static")


def spo_tracker_update(ab, ids, r, kl, kl_is_table, params, d_status):
    _check(lib().spo_tracker_update(_ptr(ab), ab.shape[0], _ptr(ids), _ptr(r), _ptr(kl), int(kl_is_table),
                                    ids.numel(), ctypes.byref(params), _ptr(d_status), _stream()),
           "spo_tracker_update")


def spo_tracker_update_repeats(ab, ids, r, kl, kl_is_table, ws, params, d_status):
    _check(lib().spo_tracker_update_repeats(_ptr(ab), ab.shape[0], _ptr(ids), _ptr(r), _ptr(kl), int(kl_is_table),
                                            ids.numel(), _ptr(ws), ws.numel() * ws.element_size(),
                                            ctypes.byref(params), _ptr(d_status), _stream()),
           "spo_tracker_update_repeats")


def spo_loss_fwd(H, W, y, logp_old, mask, cu_seqlens, a_norm, loss, logp, lse, coef, seq_sums, ws, params,
                 d_status, entropy=None):
    T, d = H.shape
    V = W.shape[0]
    S = cu_seqlens.numel() - 1
    _check(lib().spo_loss_fwd(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(logp_old), _ptr(mask),
                              _ptr(cu_seqlens), _ptr(a_norm), T, d, V, S, _ptr(loss), _ptr(logp), _ptr(lse),
                              _ptr(coef), _ptr(seq_sums), _ptr(entropy), _ptr(ws), ws.numel() * ws.element_size(),
                              ctypes.byref(params), _ptr(d_status), _stream()), "spo_loss_fwd")


def spo_loss_bwd(H, W, y, lse, coef, grad_loss, dH, dW, dW_accumulate, ws, params, d_status):
    T, d = H.shape
    V = W.shape[0]
    _check(lib().spo_loss_bwd(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(lse), _ptr(coef),
                              c_float(grad_loss), T, d, V, _ptr(dH), _dtype_code(dH), _ptr(dW),
                              int(dW_accumulate), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                              ctypes.byref(params), _ptr(d_status), _stream()), "spo_loss_bwd")


def spo_loss_fwd_bwd(H, W, y, logp_old, mask, cu_seqlens, a_norm, grad_loss, loss, logp, lse, coef, seq_sums, dH, dW,
                     dW_accumulate, ws, params, d_status, entropy=None):
    T, d = H.shape
    V = W.shape[0]
    S = cu_seqlens.numel() - 1
    _check(lib().spo_loss_fwd_bwd(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(logp_old), _ptr(mask),
                                  _ptr(cu_seqlens), _ptr(a_norm), T, d, V, S, c_float(grad_loss), _ptr(loss),
                                  _ptr(logp), _ptr(lse), _ptr(coef), _ptr(seq_sums), _ptr(entropy), _ptr(dH),
                                  _dtype_code(dH), _ptr(dW), int(dW_accumulate), _ptr(ws),
                                  ws.numel() * ws.element_size(), ctypes.byref(params), _ptr(d_status), _stream()),
           "spo_loss_fwd_bwd")


MAX_DW_SLABS = 64


def spo_dw_slab_rows(V, d, n_wanted):
    """Vocabulary-row bounds [0, ..., V] of the slabs a request for n_wanted slabs comes to (host only)."""
    buf = (c_int64 * (n_wanted + 1))()
    n = lib().spo_dw_slab_rows(V, d, n_wanted, buf)
    if n < 0:
        raise SpoError(n, "spo_dw_slab_rows")
    return [int(buf[k]) for k in range(n + 1)]


def spo_loss_fwd_bwd_slabs(H, W, y, logp_old, mask, cu_seqlens, a_norm, grad_loss, loss, logp, lse, coef, seq_sums, dH,
                           dW, dW_accumulate, ws, params, d_status, events, entropy=None):
    """spo_loss_fwd_bwd with the last dW contraction cut into len(events) slabs; `events` are
    torch.cuda.Event objects that already own a CUDA event (recorded once), one is recorded behind each slab."""
    T, d = H.shape
    V = W.shape[0]
    S = cu_seqlens.numel() - 1
    handles = (c_void_p * len(events))(*[c_void_p(ev.cuda_event) for ev in events])
    _check(lib().spo_loss_fwd_bwd_slabs(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(logp_old), _ptr(mask),
                                        _ptr(cu_seqlens), _ptr(a_norm), T, d, V, S, c_float(grad_loss), _ptr(loss),
                                        _ptr(logp), _ptr(lse), _ptr(coef), _ptr(seq_sums), _ptr(entropy), _ptr(dH),
                                        _dtype_code(dH), _ptr(dW), int(dW_accumulate), _ptr(ws),
                                        ws.numel() * ws.element_size(), ctypes.byref(params), _ptr(d_status), _stream(),
                                        len(events), handles), "spo_loss_fwd_bwd_slabs")


def dw_shards(shard_ptrs, rows_per_shard) -> SpoDwShards:
    """Shard table for spo_loss_fwd_bwd_scatter: shard_ptrs[k] is the device address (an int, or a tensor) of the
    fp32 [rows_per_shard][d] buffer that owns vocabulary rows k*rows_per_shard ..; it may be peer memory."""
    sh = SpoDwShards()
    sh.n_shards = len(shard_ptrs)
    sh.rows_per_shard = int(rows_per_shard)
    for k, ptr in enumerate(shard_ptrs):
        sh.shard[k] = ptr if isinstance(ptr, int) else ptr.data_ptr()
    return sh


def spo_loss_fwd_bwd_scatter(H, W, y, logp_old, mask, cu_seqlens, a_norm, grad_loss, loss, logp, lse, coef, seq_sums,
                             dH, dW, dW_accumulate, ws, params, d_status, shards, entropy=None):
    """spo_loss_fwd_bwd whose last dW contraction adds the finished dW into the shards that own its rows."""
    T, d = H.shape
    V = W.shape[0]
    S = cu_seqlens.numel() - 1
    _check(lib().spo_loss_fwd_bwd_scatter(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(logp_old), _ptr(mask),
                                          _ptr(cu_seqlens), _ptr(a_norm), T, d, V, S, c_float(grad_loss), _ptr(loss),
                                          _ptr(logp), _ptr(lse), _ptr(coef), _ptr(seq_sums), _ptr(entropy), _ptr(dH),
                                          _dtype_code(dH), _ptr(dW), int(dW_accumulate), _ptr(ws),
                                          ws.numel() * ws.element_size(), ctypes.byref(params), _ptr(d_status),
                                          _stream(), ctypes.byref(shards)), "spo_loss_fwd_bwd_scatter")


def spo_loss_stats(logp, logp_old, mask, cu_seqlens, a_norm, out, params):
    _check(lib().spo_loss_stats(_ptr(logp), _ptr(logp_old), _ptr(mask), _ptr(cu_seqlens), _ptr(a_norm), logp.numel(),
                                cu_seqlens.numel() - 1, _ptr(out), ctypes.byref(params), _stream()), "spo_loss_stats")


def spo_loss_mask_rows(mask, rows, d_count, ws):
    _check(lib().spo_loss_mask_rows(_ptr(mask), mask.numel(), _ptr(rows), _ptr(d_count), _ptr(ws),
                                    ws.numel() * ws.element_size(), _stream()), "spo_loss_mask_rows")


def spo_loss_fwd_bwd_rows(H, W, y, logp_old, cu_seqlens, a_norm, rows, n_listed, grad_loss, loss, logp, lse, coef,
                          seq_sums, dH, dW, dW_accumulate, ws, params, d_status):
    T, d = H.shape
    V = W.shape[0]
    S = cu_seqlens.numel() - 1
    _check(lib().spo_loss_fwd_bwd_rows(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(logp_old), _ptr(cu_seqlens),
                                       _ptr(a_norm), T, d, V, S, _ptr(rows), int(n_listed), c_float(grad_loss),
                                       _ptr(loss), _ptr(logp), _ptr(lse), _ptr(coef), _ptr(seq_sums), _ptr(dH),
                                       _dtype_code(dH), _ptr(dW), int(dW_accumulate), _ptr(ws),
                                       ws.numel() * ws.element_size(), ctypes.byref(params), _ptr(d_status),
                                       _stream()), "spo_loss_fwd_bwd_rows")


def spo_selftest_bounded_wait(limit_us, reached_end, d_status):
    _check(lib().spo_selftest_bounded_wait(int(limit_us), _ptr(reached_end), _ptr(d_status), _stream()),
           "spo_selftest_bounded_wait")


def spo_loss_active_rows(coef, rows, d_count, ws):
    _check(lib().spo_loss_active_rows(_ptr(coef), coef.numel(), _ptr(rows), _ptr(d_count), _ptr(ws),
                                      ws.numel() * ws.element_size(), _stream()), "spo_loss_active_rows")


def spo_loss_bwd_rows(H, W, y, lse, coef, grad_loss, rows, n_active, dH, dW, dW_accumulate, ws, params, d_status):
    T, d = H.shape
    V = W.shape[0]
    _check(lib().spo_loss_bwd_rows(_ptr(H), _ptr(W), _dtype_code(W), _ptr(y), _ptr(lse), _ptr(coef),
                                   c_float(grad_loss), T, d, V, _ptr(rows), int(n_active), _ptr(dH), _dtype_code(dH),
                                   _ptr(dW), int(dW_accumulate), _ptr(ws), ws.numel() * ws.element_size(),
                                   ctypes.byref(params), _ptr(d_status), _stream()), "spo_loss_bwd_rows")
