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


def mixture_runs(q0: int, q1: int) -> np.ndarray:
    """First rows of the four 16-row runs of the query mixture at key resolution (Eq. 3: "a deterministic mixture of
    recent, uniformly spaced, and boundary-adjacent positions"), ascending: the run right after the segment start, two
    runs one third and two thirds into the segment, and the last 16 rows.  A diagonal is only visible on consecutive
    rows, so the mixture is made of runs of 16 consecutive rows; the run starts are the uniformly spaced positions.
    The paper fixes neither the proportions nor the spacing: this is this build's reading."""
    units = (q1 - q0) // G_ROWS
    return np.array([q0, q0 + G_ROWS * (units // 3), q0 + G_ROWS * ((2 * units) // 3), q1 - G_ROWS], dtype=np.int64)


def probe_rows(Q: np.ndarray, K: np.ndarray, q1: int, starts=None) -> ProbeResult:
    """Probe of one head on the segment ending at q1: exact softmax rows over the causal keys, reduced per group of 16
    consecutive rows.  starts: first row of each of the four groups (default: the last 64 rows, q1 - 64 + 16 g)."""
    if starts is None:
        starts = [q1 - R_PROBE + G_ROWS * g for g in range(N_GROUPS)]
    rows = np.concatenate([np.arange(int(s0), int(s0) + G_ROWS) for s0 in starts])
    assert rows.min() >= 0 and rows.max() < q1
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


# ---------------------------------------------------------------------------------------------------------------
# Eq. 3 in its general form: r sampled query rows (a deterministic mixture of recent, uniformly spaced and
# boundary-adjacent positions) against keys pooled over blocks of width g, and the three descriptors of
# Section 3.2 (entropy, local-band concentration, agreement between the recent and the uniform group).
# The paper fixes neither the proportions of the mixture, nor how a key block that straddles the causal
# boundary is pooled, nor the formula of the agreement; the choices below are this build's reading:
#   * rows: the last r_recent rows of the segment, r_boundary rows right after the segment start, and r_uniform
#     rows spread evenly (midpoints of equal strata) over what lies between;
#   * a key block is visible to row i when its first key is <= i, and it is pooled (arithmetic mean) over its
#     visible keys only, so no future key enters a logit;
#   * agreement = 1 - total-variation distance between the two groups' mean "signatures", the signature of a row
#     being its mass re-binned into [key block 0] + [relative block offsets 0..15] + [everything else]
#     (position-independent, so rows at different depths can be compared).
SIG_LOCAL = 16


def mixture_rows(q0: int, q1: int, r_recent: int = 32, r_uniform: int = 16, r_boundary: int = 16) -> np.ndarray:
    """Row ids of the mixture, in the order recent, uniform, boundary (each ascending); all distinct."""
    span = (q1 - q0) - r_recent - r_boundary
    if span < r_uniform:
        raise ValueError("segment too short for this mixture")
    recent = np.arange(q1 - r_recent, q1)
    uniform = q0 + r_boundary + ((2 * np.arange(r_uniform) + 1) * span) // (2 * r_uniform)
    boundary = np.arange(q0, q0 + r_boundary)
    return np.concatenate([recent, uniform, boundary]).astype(np.int64)


@dataclass
class PooledProbeResult:
    A: np.ndarray          # [r, nbg] float64 softmax rows over pooled key blocks (0 on invisible blocks)
    lse: np.ndarray        # [r] float64
    colmass: np.ndarray    # [n_sub, nbg] sum over the subset's rows of A[i, kb]
    diagmass: np.ndarray   # [n_sub, nbg] sum over the subset's rows of A[i, i // g - delta], indexed by delta
    entropy: float         # mean over rows of H_i / log(max(2, visible_i)), in [0, 1]
    local_conc: float      # mean over rows of the mass of blocks whose first key is within 1024 of the row
    agreement: float       # 1 - TV(signature of subset 0, signature of subset 1); 1.0 with fewer than two subsets


def pooled_logits(Q: np.ndarray, K: np.ndarray, rows: np.ndarray, g: int, q1: int) -> np.ndarray:
    """S[t, kb] = q_i . mean(K[kb*g .. min(kb*g+g-1, i)]) / sqrt(d) for visible blocks, -inf otherwise."""
    d = Q.shape[1]
    nbg = q1 // g
    S = np.full((len(rows), nbg), -np.inf, dtype=np.float64)
    Kf = K[:q1].astype(np.float64)
    full = Kf.reshape(nbg, g, d).mean(axis=1)
    for t, i in enumerate(rows):
        q = Q[i].astype(np.float64)
        kb_d = i // g
        S[t, :kb_d] = full[:kb_d] @ q
        S[t, kb_d] = Kf[kb_d * g:i + 1].mean(axis=0) @ q
    return S * (1.0 / np.sqrt(float(d)))


def row_signature(a: np.ndarray, i: int, g: int) -> np.ndarray:
    """Mass of one probe row re-binned into [block 0] + [relative offsets 0..15] + [rest] (18 bins)."""
    sig = np.zeros(SIG_LOCAL + 2, dtype=np.float64)
    kb_d = i // g
    for kb in range(kb_d + 1):
        delta = kb_d - kb
        if delta < SIG_LOCAL:
            sig[1 + delta] += a[kb]
        elif kb == 0:
            sig[0] += a[kb]
        else:
            sig[SIG_LOCAL + 1] += a[kb]
    return sig


def pooled_probe(Q: np.ndarray, K: np.ndarray, rows: np.ndarray, g: int, q1: int, sub_bounds) -> PooledProbeResult:
    rows = np.asarray(rows, dtype=np.int64)
    S = pooled_logits(Q, K, rows, g, q1)
    mx = S.max(axis=1, keepdims=True)
    lse = mx[:, 0] + np.log(np.exp(S - mx).sum(axis=1))
    A = np.exp(S - lse[:, None])
    nbg = q1 // g
    n_sub = len(sub_bounds) - 1
    col = np.zeros((n_sub, nbg), dtype=np.float64)
    diag = np.zeros((n_sub, nbg), dtype=np.float64)
    sig = np.zeros((n_sub, SIG_LOCAL + 2), dtype=np.float64)
    ent, loc = 0.0, 0.0
    for s in range(n_sub):
        for t in range(sub_bounds[s], sub_bounds[s + 1]):
            i = int(rows[t])
            kb_d = i // g
            col[s] += A[t]
            diag[s, :kb_d + 1] += A[t, kb_d::-1]
            sig[s] += row_signature(A[t], i, g)
    for t, i in enumerate(rows):
        vis = int(i) // g + 1
        a = A[t, :vis]
        with np.errstate(divide="ignore", invalid="ignore"):
            h = -np.where(a > 0, a * np.log(a), 0.0).sum()
        ent += h / np.log(max(2, vis))
        first = np.arange(vis) * g
        loc += a[int(i) - first < LOCAL_BAND].sum()
    r = len(rows)
    agreement = 1.0
    if n_sub >= 2:
        s0 = sig[0] / max(1, sub_bounds[1] - sub_bounds[0])
        s1 = sig[1] / max(1, sub_bounds[2] - sub_bounds[1])
        agreement = 1.0 - 0.5 * float(np.abs(s0 - s1).sum())
    return PooledProbeResult(A=A, lse=lse, colmass=col, diagmass=diag, entropy=ent / r, local_conc=loc / r,
                             agreement=agreement)
