"""Oracle: the step in front of the probe -- the QKV projection of one layer with rotary position embedding, and
the side outputs the probe needs from it (64-row means of Q and K, block maxima of the squared value norms).

Test infrastructure only; never imported by the product path.

Section 3.4 lets routing run "concurrently with projection kernels or as a fused GPU reduction": the projection
is the producer of Q, K, V, so whatever the probe reduces over all keys (pooled keys, value norms) can leave the
projection's epilogue instead of being re-read.  What is computed, in float64:

    Y = X W^T                      X [n, d_model], W [(Hq + 2 Hkv) * d, d_model], heads in the order Q.., K.., V..
    Q_h = rope(Y[:, h d : (h+1) d]),  K_g = rope(Y[:, (Hq+g) d : ...]),  V_g = Y[:, (Hq+Hkv+g) d : ...]
    rope(x)[i]       = x[i] cos[t, i] - x[i + d/2] sin[t, i]           (i < d/2, token t)
    rope(x)[i + d/2] = x[i + d/2] cos[t, i] + x[i] sin[t, i]

(the "rotate half" pairing of dimension i with i + d/2 that Llama-family checkpoints use; the paper evaluates on
Llama-3.1-8B-Instruct).  cos / sin arrive as tables [n, d/2], so the oracle and the kernel rotate with the same
numbers.  Parity pins: tests/test_oracle_projection.py.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np


def rope_tables(n: int, d: int = 128, base: float = 500000.0) -> Tuple[np.ndarray, np.ndarray]:
    """cos / sin [n, d/2] float32 of the rotary embedding with inverse frequencies base^(-2 i / d)."""
    inv = base ** (-np.arange(0, d, 2, dtype=np.float64) / d)
    ang = np.arange(n, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """x [n, d] float64; cos, sin [n, d/2]."""
    h = x.shape[1] // 2
    c, s = cos.astype(np.float64), sin.astype(np.float64)
    lo, hi = x[:, :h], x[:, h:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=1)


def qkv_project(X: np.ndarray, W: np.ndarray, cos: np.ndarray, sin: np.ndarray, n_q_heads: int, n_kv_heads: int,
                d: int = 128):
    """Returns Q [Hq, n, d], K [Hkv, n, d], V [Hkv, n, d] in float64 (before any rounding)."""
    X = X.astype(np.float64)
    W = W.astype(np.float64)
    assert W.shape[0] == (n_q_heads + 2 * n_kv_heads) * d and W.shape[1] == X.shape[1]
    Y = X @ W.T
    n = X.shape[0]
    Q = np.empty((n_q_heads, n, d)); K = np.empty((n_kv_heads, n, d)); V = np.empty((n_kv_heads, n, d))
    for h in range(n_q_heads):
        Q[h] = rope(Y[:, h * d:(h + 1) * d], cos, sin)
    for g in range(n_kv_heads):
        K[g] = rope(Y[:, (n_q_heads + g) * d:(n_q_heads + g + 1) * d], cos, sin)
        V[g] = Y[:, (n_q_heads + n_kv_heads + g) * d:(n_q_heads + n_kv_heads + g + 1) * d]
    return Q, K, V


def block_means(X: np.ndarray, block: int = 64) -> np.ndarray:
    """[n, d] -> [n / block, d]: arithmetic mean of every run of `block` rows."""
    n, d = X.shape
    return X.astype(np.float64).reshape(n // block, block, d).mean(axis=1)


def block_max_sq_norm(V: np.ndarray, block: int = 64) -> np.ndarray:
    """[n, d] -> [n / block]: max over the block's rows of ||v||_2^2."""
    n, d = V.shape
    return (V.astype(np.float64) ** 2).sum(axis=1).reshape(n // block, block).max(axis=1)
