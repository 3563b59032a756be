"""Host-side analysis of calibration results (numpy only; the scores themselves come from the CUDA
calibration kernels through heatkv_calibrate_scores / heatkv_finalize_scores)."""
from __future__ import annotations

import numpy as np

__all__ = ["scas_rank_dispersion"]


def scas_rank_dispersion(scas_runs: np.ndarray, s: int) -> np.ndarray:
    """Rank stability of the S-CAS head ordering over R calibration runs (paper appendix on S-CAS stability).

    scas_runs: [R, L, H, K].  For every prunable source scale (0-based s <= k <= K-2) the heads are ranked
    per run by ascending S-CAS (ties by head index, as the schedule builder does); the result is, per scale,
    the mean over heads of the standard deviation of a head's rank around its own mean rank.  [K] float64."""
    runs = np.asarray(scas_runs, dtype=np.float64)
    R, L, H, K = runs.shape
    flat = runs.reshape(R, L * H, K)
    order = np.argsort(flat, axis=1, kind="stable")                  # [R, T, K]: heads by ascending score
    ranks = np.empty_like(order)
    r_idx, k_idx = np.meshgrid(np.arange(R), np.arange(K), indexing="ij")
    ranks[r_idx[:, None, :], order, k_idx[:, None, :]] = np.arange(L * H)[None, :, None]
    disp = ranks.astype(np.float64).std(axis=0).mean(axis=0)          # std over runs, mean over heads
    out = np.zeros(K, dtype=np.float64)
    out[s:K - 1] = disp[s:K - 1]
    return out
