"""Threshold calibration to a target density (the paper fixes its thresholds offline so that a calibration set
reaches a target budget, Sec. 4.4 and the calibration-cost table of the supplementary system analysis).

Density is non-increasing in each threshold (App. D.3), so a bisection on a common scale factor applied to
(alpha_base, alpha_rescue) finds the pair that realises a wanted density on given inputs.  The density of every
probe comes from the library's selector; nothing is computed here beyond the bisection itself.
"""
from __future__ import annotations

from typing import Callable, Tuple


def bisect_alpha(density_of: Callable[[float, float], float], target: float, ratio: float = 0.18 / 0.22,
                 lo: float = 1e-4, hi: float = 1.0, iters: int = 18, tol: float = 1e-4) -> Tuple[float, float, float]:
    """Finds alpha_base in [lo, hi] (alpha_rescue = ratio * alpha_base, capped at 1) whose mean density is closest to
    `target`.  `density_of(alpha_base, alpha_rescue)` must be non-increasing in both arguments.
    Returns (alpha_base, alpha_rescue, density)."""
    def pair(a):
        return a, min(1.0, ratio * a)

    d_lo = density_of(*pair(lo))     # loosest thresholds: highest density
    d_hi = density_of(*pair(hi))     # tightest: lowest density (forced blocks remain)
    if target >= d_lo:
        return (*pair(lo), d_lo)
    if target <= d_hi:
        return (*pair(hi), d_hi)
    best = (abs(d_lo - target), lo, d_lo)
    a, b = lo, hi
    for _ in range(iters):
        mid = (a * b) ** 0.5          # thresholds act on a ratio scale
        d = density_of(*pair(mid))
        if abs(d - target) < best[0]:
            best = (abs(d - target), mid, d)
        if abs(d - target) <= tol:
            break
        if d > target:
            a = mid
        else:
            b = mid
    return (*pair(best[1]), best[2])


def calibrate_on_gpu(Q, stats, block: int, target: float, n_sink: int = 1, n_local: int = 1, n_recent: int = 1,
                     ratio: float = 0.18 / 0.22, **kw):
    """Bisection with the CUDA selector as the density probe.  Q: [L,N,Hq,d] bf16 on the GPU, stats from
    rbs_block_stats.  Returns (alpha_base, alpha_rescue, mean density)."""
    import torch

    from .binding import RBS_OP_SELECT, RbsShape, rbs_select, workspace_bytes
    L, N, Hq, d = Q.shape
    M = (N + block - 1) // block
    shape = RbsShape(L, N, Hq, stats.centroid.shape[1], d, block)
    mask = torch.empty(L, Hq, M, (M + 31) // 32, dtype=torch.int32, device=Q.device)
    dens = torch.empty(L, Hq, dtype=torch.float32, device=Q.device)
    ws = torch.empty(max(256, workspace_bytes(RBS_OP_SELECT, shape)), dtype=torch.uint8, device=Q.device)

    def density_of(ab, ar):
        rbs_select(Q, stats, block, ab, ar, n_sink, n_local, n_recent, mask=mask, density=dens, workspace=ws)
        return float(dens.mean().item())

    return bisect_alpha(density_of, target, ratio=ratio, **kw)
