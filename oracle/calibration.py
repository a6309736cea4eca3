"""Oracle: offline calibration of Section 3.5 and the calibrated predictor e of Eq. 4, float64.

Test infrastructure only; never imported by the product path.

The paper states what calibration produces (a one-sided residual quantile delta_q of the probe's mass estimate, the
coverage of the resulting empirical certificate, and "a small monotone regressor" e fed by probe descriptors and
candidate metadata) but no formulas.  This build's reading, restated here from its definitions:
  * residual of one (head, candidate): r = m_hat - m_true, with m_true the mean over all audited rows of the exactly
    retained mass exp(lse_sel - lse_full);  delta_q = the smallest residual value d such that at least a fraction q
    of the residuals is <= d, and never negative (one-sided: only over-estimates are corrected);
  * the empirical certificate of a head is 2 (1 - max(0, m_hat - delta_q)) V_max (Eq. 5 with the lower-confidence
    mass); it "covers" when the head's mean row error ||O_dense - O_sparse|| is not larger;
  * e = step(z), z = sum_k w_k f_k over the six features (1 - m_hat, u, entropy, 1 - local, 1 - agreement,
    1 - pairs / dense pairs), w >= 0, step = isotonic (non-decreasing) least-squares fit of the observed error on z.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from .patterns import DENSE, Candidate, m_hat_from_fx


def one_sided_quantile(residuals: Sequence[float], q: float) -> float:
    """Smallest d >= 0 such that at least ceil(q * N) of the residuals are <= d."""
    r = np.sort(np.asarray(residuals, dtype=np.float64))
    if len(r) == 0:
        return 0.0
    k = int(np.ceil(q * len(r)))
    k = min(max(k, 1), len(r))
    return max(0.0, float(r[k - 1]))


def true_mass(lse_sel: np.ndarray, lse_full: np.ndarray) -> float:
    """Mean over rows of the exactly retained mass min(1, exp(lse_sel - lse_full))."""
    return float(np.minimum(1.0, np.exp(lse_sel.astype(np.float64) - lse_full.astype(np.float64))).mean())


def certificate_covers(m_hat: float, delta_q: float, vmax: float, mean_err: float) -> bool:
    return mean_err <= 2.0 * (1.0 - max(0.0, m_hat - delta_q)) * float(np.float32(vmax))


def isotonic_fit(z: Sequence[float], y: Sequence[float]) -> Tuple[np.ndarray, np.ndarray]:
    """Non-decreasing least-squares step function of y on z by pooling adjacent violators.

    Returns (bp_z, bp_e): the function equals bp_e[k] on [bp_z[k], bp_z[k+1]) and 0 below bp_z[0].  Ties in z are
    merged first (their mean y, weight = count)."""
    z = np.asarray(z, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    order = np.argsort(z, kind="stable")
    z, y = z[order], y[order]
    blocks: List[List[float]] = []        # [z_first, sum_y, weight]
    i = 0
    while i < len(z):
        j = i
        while j + 1 < len(z) and z[j + 1] == z[i]:
            j += 1
        blocks.append([float(z[i]), float(y[i:j + 1].sum()), float(j - i + 1)])
        i = j + 1
    merged: List[List[float]] = []
    for b in blocks:
        merged.append(b)
        while len(merged) >= 2 and merged[-2][1] / merged[-2][2] > merged[-1][1] / merged[-1][2]:
            hi = merged.pop()
            merged[-1][1] += hi[1]
            merged[-1][2] += hi[2]
    return (np.array([b[0] for b in merged], dtype=np.float64),
            np.array([b[1] / b[2] for b in merged], dtype=np.float64))


def step_eval(bp_z: np.ndarray, bp_e: np.ndarray, z: float) -> float:
    e = 0.0
    for k in range(len(bp_z)):
        if bp_z[k] <= z:
            e = float(bp_e[k])
    return e


def features(cov_fx: np.ndarray, pairs: int, descr: Sequence[float], q0: int, q1: int) -> List[float]:
    """The six regressor inputs of one (item, candidate); descr = (entropy, local, agreement) as float32 values."""
    m_hat, u = m_hat_from_fx(cov_fx)
    dense_pairs = float((q1 * (q1 + 1) - q0 * (q0 + 1)) // 2)
    return [1.0 - m_hat, u, float(np.float32(descr[0])), 1.0 - float(np.float32(descr[1])),
            1.0 - float(np.float32(descr[2])), 1.0 - float(int(pairs)) / dense_pairs]


def regressor_eval(lib: List[Candidate], cov_fx: np.ndarray, pairs: np.ndarray, descr: np.ndarray,
                   seg_of_item: Sequence[Tuple[int, int]], w: Sequence[float], bp_z: np.ndarray, bp_e: np.ndarray):
    """e[item][c] for every item and candidate (0 for dense): z accumulated left to right, one rounding per operation."""
    n_items, n_cand = cov_fx.shape[0], len(lib)
    e = np.zeros((n_items, n_cand), dtype=np.float64)
    for it in range(n_items):
        q0, q1 = seg_of_item[it]
        for c, cand in enumerate(lib):
            if cand.pattern == DENSE:
                continue
            f = features(cov_fx[it, c], int(pairs[it, c]), descr[it], q0, q1)
            z = 0.0
            for k in range(6):
                z = z + float(w[k]) * f[k]
            e[it, c] = step_eval(bp_z, bp_e, z)
    return e
