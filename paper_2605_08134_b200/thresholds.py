"""Layer-wise threshold allocation (Sec. 3.1, "Reuse rate allocation"): offline calibration, host-side only.

From per-layer samples of the drift score (as `dare_layer_last_selection` / `dare_drift_scores` return them on a
calibration run):
    s_l   = mean over steps and tokens of the drift score of layer l                       (Eq. 1)
    phi_l = (L * phi_bar) * softmax(-s / eps)_l,  clipped to [0, 1]                         (allocation rule)
    tau_l = the phi_l-quantile of layer l's drift scores                                    (threshold)
so that layers with less drift get a larger share of the reuse budget.  The clip is this library's reading: the
paper does not say what happens when a layer's share exceeds 1.
"""
from __future__ import annotations

import numpy as np


def layer_drift_scores(samples) -> np.ndarray:
    """Eq. 1: one mean per layer.  `samples`: sequence of L arrays of finite drift scores."""
    return np.array([float(np.mean(np.asarray(s, np.float64))) for s in samples])


def reuse_quantiles(s, phi_bar: float, eps: float) -> np.ndarray:
    s = np.asarray(s, np.float64)
    z = -s / eps
    z = z - z.max()
    sm = np.exp(z) / np.exp(z).sum()
    return np.clip(len(s) * phi_bar * sm, 0.0, 1.0)


def thresholds(samples, phi_bar: float = 0.3, eps: float = 0.1):
    """-> (tau [L], phi [L], s [L]).  tau_l is the phi_l-quantile (linear interpolation between order statistics)."""
    s = layer_drift_scores(samples)
    phi = reuse_quantiles(s, phi_bar, eps)
    tau = np.array([float(np.quantile(np.asarray(x, np.float64), p)) for x, p in zip(samples, phi)])
    return tau, phi, s
