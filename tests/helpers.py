"""Shared helpers for the GPU parity tests: upload inputs, call the C-ABI binding, fetch results."""

import numpy as np


def rel_fro(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.linalg.norm(want)
    return np.linalg.norm(got - want) / (den if den > 0 else 1.0)


def worst_row_tile_error(got, want, tile=256, floor_share=0.05):
    """Largest relative Frobenius error over consecutive row tiles of a matrix (a whole-matrix norm
    hides one wrong tile among hundreds).  Tiles whose reference norm is below floor_share x the
    median tile norm carry (almost) no signal and are left out.  Returns (worst, checked, n_tiles,
    last_tile_checked)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    rows = want.shape[0]
    n_tiles = -(-rows // tile)
    norms = np.array([np.linalg.norm(want[i * tile:(i + 1) * tile]) for i in range(n_tiles)])
    floor = floor_share * np.median(norms)
    worst, checked = 0.0, 0
    for i in range(n_tiles):
        if norms[i] < floor or norms[i] == 0.0:
            continue
        sl = slice(i * tile, min((i + 1) * tile, rows))
        worst = max(worst, np.linalg.norm(got[sl] - want[sl]) / norms[i])
        checked += 1
    return worst, checked, n_tiles, bool(norms[-1] >= floor and norms[-1] > 0.0)


def dev(x, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t if dtype is None else t.to(dtype)


def status_word():
    import torch
    return torch.zeros(4, dtype=torch.int32, device="cuda")


def ws_bytes(which, **kw):
    import torch
    from paper_2509_13232_b200 import binding as B
    n = B.spo_workspace_bytes(which, **kw)
    return torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")


def run_loss(lb, params=None, grad_loss=1.0, dh_bf16=None, want_seq_sums=True, dw_init=None, mask_none=False,
             one_pass=False, want_entropy=False):
    """Forward + backward through the binding for a LossBatch; returns numpy outputs.
    one_pass: a single spo_loss_fwd_bwd call instead of spo_loss_fwd followed by spo_loss_bwd."""
    import torch
    from paper_2509_13232_b200 import binding as B
    params = params or B.default_params()
    tdt = torch.bfloat16 if lb.bf16 else torch.float32
    H, W = dev(lb.h, tdt), dev(lb.w, tdt)
    T, d = H.shape
    V = W.shape[0]
    S = len(lb.cu_seqlens) - 1
    y, lo = dev(lb.y), dev(lb.logp_old)
    mask = None if mask_none else dev(lb.mask)
    cu, an = dev(lb.cu_seqlens), dev(lb.a_norm)
    f32 = dict(dtype=torch.float32, device="cuda")
    loss = torch.zeros(4, **f32)
    logp, lse, coef = (torch.full((max(T, 1),), float("nan"), **f32) for _ in range(3))
    seq = torch.zeros((max(S, 1), 3), **f32) if want_seq_sums else None
    st = status_word()
    ent = torch.full((max(T, 1),), float("nan"), **f32) if want_entropy else None
    if dh_bf16 is None:
        dh_bf16 = lb.bf16
    dH = torch.full((max(T, 1), d), float("nan"), dtype=torch.bfloat16 if dh_bf16 else torch.float32, device="cuda")
    if dw_init is None:
        dW = torch.full((V, d), float("nan"), **f32)
        acc = 0
    else:
        dW = dev(dw_init).clone()
        acc = 1
    if one_pass:
        ws = ws_bytes(B.WS_LOSS_FWD_BWD, T=T, d=d, V=V, B=S)
        B.spo_loss_fwd_bwd(H, W, y, lo, mask, cu, an, grad_loss, loss, logp, lse, coef, seq, dH[:T], dW, acc, ws,
                           params, st, entropy=ent)
    else:
        wsf = ws_bytes(B.WS_LOSS_FWD, T=T, d=d, V=V, B=S)
        B.spo_loss_fwd(H, W, y, lo, mask, cu, an, loss, logp, lse, coef, seq, wsf, params, st, entropy=ent)
        wsb = ws_bytes(B.WS_LOSS_BWD, T=T, d=d, V=V)
        B.spo_loss_bwd(H, W, y, lse, coef, grad_loss, dH, dW, acc, wsb, params, st)
    torch.cuda.synchronize()
    return {
        "loss": float(loss[0].item()), "logp": logp[:T].cpu().numpy(), "lse": lse[:T].cpu().numpy(),
        "coef": coef[:T].cpu().numpy(), "seq_sums": None if seq is None else seq[:S].cpu().numpy(),
        "dH": dH[:T].float().cpu().numpy(), "dW": dW.cpu().numpy(), "status": int(st[0].item()),
        "entropy": None if ent is None else ent[:T].cpu().numpy(),
    }


def oracle_loss(lb, params=None, grad_loss=1.0, mask_none=False):
    from oracle import spo_oracle as O
    clip_lo = 0.2 if params is None else float(np.float32(params.clip_lo))
    clip_hi = 0.28 if params is None else float(np.float32(params.clip_hi))
    mask = None if mask_none else lb.mask
    agg = 0 if params is None else int(params.agg_mode)
    sur = 0 if params is None else int(params.surrogate)
    dual = None if params is None or params.dual_clip == 0.0 else float(np.float32(params.dual_clip))
    fwd = O.loss_forward(lb.h, lb.w, lb.y, lb.logp_old, mask, lb.cu_seqlens, lb.a_norm, clip_lo, clip_hi, agg, sur,
                         dual)
    dh, dw = O.loss_backward(lb.h, lb.w, lb.y, fwd["lse"], fwd["coef"], grad_loss)
    fwd["dH"], fwd["dW"] = dh, dw
    return fwd
