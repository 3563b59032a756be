"""Analysis of calibration results: a binding only -- the arithmetic is heatkv_rank_dispersion in the C library
(the scores themselves come from the CUDA calibration kernels through heatkv_calibrate_scores /
heatkv_finalize_scores)."""
from __future__ import annotations

import numpy as np

from .heatkv import heatkv_rank_dispersion

__all__ = ["scas_rank_dispersion"]


def scas_rank_dispersion(scas_runs: np.ndarray, s: int) -> np.ndarray:
    """Rank stability of the S-CAS head ordering over R calibration runs (paper appendix on S-CAS stability).

    scas_runs: [R, L, H, K].  Per prunable source scale (0-based s <= k <= K-2): mean over heads of the standard
    deviation of a head's rank position around its own mean rank.  [K] float64."""
    return heatkv_rank_dispersion(scas_runs, s)
