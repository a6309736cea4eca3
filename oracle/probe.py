"""Oracle: the shared attention probe (Eq. 3, Section 3.2) in the last-64-query form, float64.

Test infrastructure only; never imported by the product path.

Eq. 3 scores r sampled queries against pooled keys.  The form built here fixes I = the last 64
query rows of the segment and key pooling width 1 for the column / diagonal signal (the paper's
"recent queries" signal for vertical-slash), and pools both queries and keys over 64-row blocks
(arithmetic mean) for the coarse block signal.  The probe rows are soft-maxed so that "mass" is
defined; block scores stay raw pooled logits (a per-row top-k does not change under softmax).
No normalisation by the number of contributing rows is applied to vert / slash.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

from .attention import causal_logits

B = 64
R_PROBE = 64
N_GROUPS = 4
G_ROWS = R_PROBE // N_GROUPS
LOCAL_BAND = 1024


@dataclass
class ProbeResult:
    vert: np.ndarray        # [4, q1] float32: vert[g, j] = sum_{i in I_g} P[i, j]
    slash: np.ndarray       # [4, q1] float32: slash[g, o] = sum_{i in I_g, i-o>=0} P[i, i-o]
    lse: np.ndarray         # [64] float32: log-sum-exp of each probe row
    P: np.ndarray           # [64, q1] float64: the probe rows themselves (not a product output)
    entropy: float          # mean over probe rows of -sum_j P log P
    local_conc: float       # mean over probe rows of the mass with i - j < 1024


def probe_rows(Q: np.ndarray, K: np.ndarray, q1: int) -> ProbeResult:
    """Probe of one head on the segment ending at q1: exact softmax rows q1-64 .. q1-1 over keys [0, q1)."""
    rows = np.arange(q1 - R_PROBE, q1)
    l = causal_logits(Q, K, rows, q1)
    mx = l.max(axis=1, keepdims=True)
    lse = mx[:, 0] + np.log(np.exp(l - mx).sum(axis=1))
    P = np.exp(l - lse[:, None])                      # 0 where j > i
    vert = P.reshape(N_GROUPS, G_ROWS, q1).sum(axis=1)
    slash = np.zeros((N_GROUPS, q1), dtype=np.float64)
    for t, i in enumerate(rows):                      # P[i, i-o] for o = 0..i  is the reversed causal part
        slash[t // G_ROWS, :i + 1] += P[t, i::-1]
    with np.errstate(divide="ignore", invalid="ignore"):
        plogp = np.where(P > 0, P * np.log(P), 0.0)
    entropy = float(-plogp.sum(axis=1).mean())
    j = np.arange(q1)[None, :]
    local = float((P * (rows[:, None] - j < LOCAL_BAND)).sum(axis=1).mean())
    return ProbeResult(vert=vert.astype(np.float32), slash=slash.astype(np.float32),
                       lse=lse.astype(np.float32), P=P, entropy=entropy, local_conc=local)


def pool_mean(X: np.ndarray, n_rows: Optional[int] = None) -> np.ndarray:
    """Arithmetic mean of consecutive 64-row blocks: [n, d] -> [n/64, d] float64."""
    n_rows = X.shape[0] if n_rows is None else n_rows
    return X[:n_rows].reshape(n_rows // B, B, X.shape[1]).mean(axis=1)


def block_scores(Q: np.ndarray, K: np.ndarray, q0: int, q1: int) -> np.ndarray:
    """bscore[qb - q0/64, kb] = (qpool[qb] . kpool[kb]) / sqrt(d) for kb <= qb, -inf above; float32."""
    d = Q.shape[1]
    qp = pool_mean(Q, q1)[q0 // B:]
    kp = pool_mean(K, q1)
    s = (qp @ kp.T) * (1.0 / np.sqrt(float(d)))
    qb = np.arange(q0 // B, q1 // B)[:, None]
    kb = np.arange(q1 // B)[None, :]
    s[kb > qb] = -np.inf
    return s.astype(np.float32)


def value_norms(V: np.ndarray, q1: int):
    """vnorm[j] = ||v_j||_2 for j < q1 and their maximum V_max (Eq. 5), float32."""
    vn = np.sqrt((V[:q1] * V[:q1]).sum(axis=1))
    return vn.astype(np.float32), np.float32(vn.max())
