"""Oracle: the attention-output error certificate of Eq. 5, float64.

Test infrastructure only; never imported by the product path.

For one exact attention row a with retained set S of mass m, and a~ the renormalisation of a on S:
||aV - a~V||_2 <= 2 (1 - m) V_max.  When the log-sum-exp of a row is known both over the selected
keys (lse_sel) and over all causal keys (lse_full), the retained mass is exactly
m = exp(lse_sel - lse_full).
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np


def row_mass(lse_sel: np.ndarray, lse_full: np.ndarray) -> np.ndarray:
    """m_i = min(1, exp(lse_sel_i - lse_full_i))."""
    return np.minimum(1.0, np.exp(lse_sel.astype(np.float64) - lse_full.astype(np.float64)))


def certificate(lse_sel: np.ndarray, lse_full: np.ndarray, vmax: float, onorm: Optional[np.ndarray] = None,
                delta_q: float = 0.0) -> Tuple[np.ndarray, np.ndarray, Optional[np.ndarray], float, float, float]:
    """Eq. 5 per row and per head.

    Returns (m_row, cert_row, cert_tight_row, m_head, cert_head, cert_head_max):
      cert_row_i   = 2 (1 - m_i) V_max                        (Eq. 5)
      cert_tight_i = (1 - m_i) (V_max + ||O~_i||)              (same derivation, keeps the -(1-m) O~ term exact)
      m_head       = mean_i m_i,  m_low = max(0, m_head - delta_q),  cert_head = 2 (1 - m_low) V_max
      cert_head_max = max_i cert_row_i
    """
    vmax = float(np.float32(vmax))
    m = row_mass(lse_sel, lse_full)
    cert = 2.0 * (1.0 - m) * vmax
    tight = None if onorm is None else (1.0 - m) * (vmax + onorm.astype(np.float64))
    m_head = float(m.mean())
    m_low = max(0.0, m_head - delta_q)
    return m, cert, tight, m_head, 2.0 * (1.0 - m_low) * vmax, float(cert.max())
