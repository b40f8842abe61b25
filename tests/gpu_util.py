"""Shared helpers of the GPU parity tests: run the CUDA path through the binding, run the oracle on the
same bytes, compare.  Tolerances are the ones the target states: scores 1e-4 relative (absolute floor
1e-6), decisions / indices / codes bit-exact except tokens whose score lies within 1e-4 relative of a
threshold, dequantised K/V within 1e-3 absolute."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2602_14236_b200 import binding as sc

SCORE_RTOL = 1e-4
SCORE_ATOL = 1e-6
NEAR_RTOL = 1e-4


def oracle_params(p: sc.Params) -> oracle.Params:
    return oracle.Params(patch=p.patch, pyr_levels=p.pyr_levels, poly_n=p.poly_n, poly_sigma=p.poly_sigma, win=p.win,
                         iters=p.iters, eps_det=p.eps_det, canny_lo=p.canny_lo, canny_hi=p.canny_hi,
                         var_radius=p.var_radius, sigma_ref=p.sigma_ref, w_edge=p.w_edge, w_color=p.w_color,
                         tau_t=p.tau_t, theta_R=p.theta_R, tau_high=p.tau_high, tau_med=p.tau_med,
                         tau_low=p.tau_low, patch_reuse=p.patch_reuse, color_norm=p.color_norm,
                         color_kappa=p.color_kappa, color_sigma_min=p.color_sigma_min)


def assert_scores_close(gpu: np.ndarray, ref: np.ndarray, what: str):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    err = np.abs(gpu - ref)
    bound = SCORE_ATOL + SCORE_RTOL * np.abs(ref)
    bad = err > bound
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} beyond tolerance, worst {err.max():.3e} " \
                          f"(ref {ref.ravel()[np.argmax(err)]:.6g})"


def gpu_scores(ctx: sc.Context, frames_np: np.ndarray, want_flow: bool = False):
    """frames [T][H][W][3] uint8 -> (dP [T][n_tok] float32 with row 0 unused, s [T][n_tok] float32[, flow])."""
    import torch
    T = frames_np.shape[0]
    fr = torch.from_numpy(frames_np).cuda()
    dP = torch.zeros((T, ctx.n_tok), dtype=torch.float32, device="cuda")
    s = torch.zeros((T, ctx.n_tok), dtype=torch.float32, device="cuda")
    H, W = frames_np.shape[1:3]
    fl = torch.zeros((max(T - 1, 1), 2, H, W), dtype=torch.float64, device="cuda") if want_flow else None
    if T > 1:
        sc.salicache_flow_score(ctx, fr[:-1], fr[1:], T - 1, dP[1:], fl)
    sc.salicache_saliency(ctx, fr, T, s)
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0
    out = (dP.cpu().numpy(), s.cpu().numpy())
    return out + (fl.cpu().numpy(),) if want_flow else out


def gpu_select(ctx: sc.Context, dP: np.ndarray, s: np.ndarray, first_has_no_prev: bool = True, fill0=(0, 0, 0)):
    import torch
    T, n = s.shape
    d_dP = torch.from_numpy(np.ascontiguousarray(dP, np.float32)).cuda() if dP is not None else None
    d_s = torch.from_numpy(np.ascontiguousarray(s, np.float32)).cuda()
    out = dict(
        decision=torch.full((T, n), 255, dtype=torch.uint8, device="cuda"),
        idx=torch.full((T, 3, n), -7, dtype=torch.int32, device="cuda"),
        counts=torch.full((T, 5), -1, dtype=torch.int32, device="cuda"),
        redundant=torch.full((T,), 255, dtype=torch.uint8, device="cuda"),
        row_offset=torch.full((T, 3), -1, dtype=torch.int64, device="cuda"),
        fill=torch.tensor(list(fill0), dtype=torch.int64, device="cuda"),
    )
    sc.salicache_select(ctx, d_dP, d_s, T, first_has_no_prev, out["decision"], out["idx"], out["counts"],
                        out["redundant"], out["row_offset"], out["fill"])
    torch.cuda.synchronize()
    return out


def oracle_select_all(dP: np.ndarray, s: np.ndarray, p: oracle.Params, first_has_no_prev: bool = True):
    T, n = s.shape
    dec = np.empty((T, n), np.uint8)
    idx = np.empty((T, 3, n), np.int32)
    counts = np.empty((T, 5), np.int32)
    red = np.empty(T, np.uint8)
    for t in range(T):
        has_prev = dP is not None and not (first_has_no_prev and t == 0)
        dec[t], idx[t], counts[t], red[t], _ = oracle.select(dP[t] if dP is not None else None, s[t], has_prev, p)
    off, _ = oracle.row_offsets(counts)
    return dec, idx, counts, red, off


def near_threshold(dP: np.ndarray, s: np.ndarray, p: oracle.Params) -> np.ndarray:
    """Tokens whose score lies within 1e-4 relative of a threshold it is compared with."""
    near = np.zeros(s.shape, bool)
    for tau in (p.tau_high, p.tau_med, p.tau_low):
        near |= np.abs(s - tau) <= NEAR_RTOL * abs(tau)
    if dP is not None:
        near |= np.abs(dP - p.tau_t) <= NEAR_RTOL * abs(p.tau_t)
    return near
