"""Oracle: dense causal attention (Eq. 1) and masked attention (Section 2.1), float64.

Test infrastructure only; never imported by the product path.

Inputs are float64 arrays holding the exact values of the bf16 inputs.  Every query row is
computed by the plain definition: all causal logits of the row, their maximum, exponentials,
the normaliser and the weighted sum of value rows.  Rows are handled a few at a time only to
bound memory; no row's arithmetic depends on the chunking.
"""
from __future__ import annotations

from typing import Callable, Iterable, Optional, Tuple

import numpy as np


def _row_chunks(rows: np.ndarray, chunk: int) -> Iterable[np.ndarray]:
    for s in range(0, len(rows), chunk):
        yield rows[s:s + chunk]


def causal_logits(Q: np.ndarray, K: np.ndarray, rows: np.ndarray, n_keys: Optional[int] = None) -> np.ndarray:
    """l[i, j] = (Q_i . K_j) / sqrt(d) for the given rows and keys [0, n_keys); j > i is set to -inf.

    Eq. 1: the additive causal mask C is 0 for j <= i and -inf otherwise.
    """
    d = Q.shape[1]
    n_keys = K.shape[0] if n_keys is None else n_keys
    l = (Q[rows] @ K[:n_keys].T) * (1.0 / np.sqrt(float(d)))
    j = np.arange(n_keys)[None, :]
    l[j > rows[:, None]] = -np.inf
    return l


def dense_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, rows: Optional[np.ndarray] = None,
                    chunk: int = 256) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1: O = softmax(Q K^T / sqrt(d) + C) V for one head.

    Returns (O[len(rows), d] float32, lse[len(rows)] float32) with lse_i = log sum_j exp(l_ij).
    """
    n = Q.shape[0]
    rows = np.arange(n) if rows is None else np.asarray(rows)
    O = np.empty((len(rows), V.shape[1]), dtype=np.float32)
    lse = np.empty(len(rows), dtype=np.float32)
    at = 0
    for r in _row_chunks(rows, chunk):
        nk = int(r.max()) + 1
        l = causal_logits(Q, K, r, nk)
        mx = l.max(axis=1, keepdims=True)
        p = np.exp(l - mx)
        L = p.sum(axis=1, keepdims=True)
        O[at:at + len(r)] = ((p @ V[:nk]) / L).astype(np.float32)
        lse[at:at + len(r)] = (mx[:, 0] + np.log(L[:, 0])).astype(np.float32)
        at += len(r)
    return O, lse


def attention_matrix(Q: np.ndarray, K: np.ndarray) -> np.ndarray:
    """The full n x n matrix A of Eq. 1 (small n only)."""
    n = Q.shape[0]
    l = causal_logits(Q, K, np.arange(n))
    mx = l.max(axis=1, keepdims=True)
    p = np.exp(l - mx)
    return p / p.sum(axis=1, keepdims=True)


def masked_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray,
                     mask_rows: Callable[[np.ndarray, int], np.ndarray],
                     rows: Optional[np.ndarray] = None, chunk: int = 256
                     ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Section 2.1: logits outside the binary mask M become -inf and the softmax renormalises.

    mask_rows(rows, n_keys) returns the boolean rows of M (True = selected) for keys [0, n_keys);
    causality is applied on top of it.  Returns float32 (O~, lse_sel, onorm) where
    lse_sel_i = log sum_{j in M_i} exp(l_ij) and onorm_i = ||O~_i||_2.
    Every pattern of the library keeps the diagonal, so no row is empty.
    """
    n = Q.shape[0]
    rows = np.arange(n) if rows is None else np.asarray(rows)
    O = np.empty((len(rows), V.shape[1]), dtype=np.float32)
    lse = np.empty(len(rows), dtype=np.float32)
    onorm = np.empty(len(rows), dtype=np.float32)
    at = 0
    for r in _row_chunks(rows, chunk):
        nk = int(r.max()) + 1
        l = causal_logits(Q, K, r, nk)
        M = mask_rows(r, nk)
        l[~M] = -np.inf
        mx = l.max(axis=1, keepdims=True)
        p = np.exp(l - mx)
        L = p.sum(axis=1, keepdims=True)
        o = (p @ V[:nk]) / L
        O[at:at + len(r)] = o.astype(np.float32)
        lse[at:at + len(r)] = (mx[:, 0] + np.log(L[:, 0])).astype(np.float32)
        onorm[at:at + len(r)] = np.sqrt((o * o).sum(axis=1)).astype(np.float32)
        at += len(r)
    return O, lse, onorm


def relative_error(O: np.ndarray, O_tilde: np.ndarray, eps: float = 1e-12) -> float:
    """Eq. 9: E_rel = ||O - O~||_F / (||O||_F + eps)."""
    O = O.astype(np.float64)
    O_tilde = O_tilde.astype(np.float64)
    return float(np.linalg.norm(O - O_tilde) / (np.linalg.norm(O) + eps))
