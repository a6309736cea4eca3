"""Oracle: the pattern library of Section 3.1 -- masks, index estimation, pair counts, coverage.

Test infrastructure only; never imported by the product path.

Patterns (Section 2.1 / 3.1): A-shape (initial + local tokens), vertical-slash (content dependent
columns and diagonals), block-sparse (coarse 64 x 64 query-key blocks), dense.  The paper fixes the
families and which probe signal scores each ("recent queries score global columns and diagonals,
pooled queries and keys score coarse blocks"); it gives no tie-break, no budget units and no
executed form of a slash.  The readings taken here:
  * ranking keys are integers: fx(x) = floor(x * 2^32) of the fp32 probe mass, summed over the four
    probe groups; order is key descending, then index ascending;
  * vertical-slash keeps offset 0 (the diagonal) inside its slash budget;
  * the executed ("BLOCK") form of a slash set S is the set D of 64-aligned block diagonals the
    slashes touch, D = {floor(o/64), ceil(o/64) : o in S}; STRICT keeps token-exact diagonals;
  * block-sparse always keeps the diagonal block inside its budget;
  * a segment [q0, q1) applies its mask to query rows [q0, q1) against keys [0, q1).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Tuple

import numpy as np

DENSE, A_SHAPE, VERTICAL_SLASH, BLOCK_SPARSE = 0, 1, 2, 3
B = 64                 # block edge
R_PROBE = 64           # probe rows
N_GROUPS = 4           # probe row groups of 16
FX_ONE = 1 << 32       # fixed-point unit


@dataclass(frozen=True)
class Candidate:
    pattern: int
    b0: int = 0        # A: n_sink | VS: k_v | BS: k_b
    b1: int = 0        # A: window | VS: k_s
    strict: bool = False   # VS only: token-exact diagonals instead of block diagonals


@dataclass
class IndexSet:
    """Indices of one (segment, head, candidate)."""
    cand: Candidate
    q0: int
    q1: int
    V: Optional[np.ndarray] = None      # VS: vertical key indices, ascending
    S: Optional[np.ndarray] = None      # VS: slash offsets, ascending
    D: Optional[np.ndarray] = None      # VS: block-diagonal deltas, ascending
    blk: Optional[List[np.ndarray]] = None   # BS: per query block of the segment, ascending key blocks


# ----------------------------------------------------------------------------- fixed point + top-k
def fx(x: np.ndarray) -> np.ndarray:
    """floor(x * 2^32) of non-negative fp32 values, as uint64 (exact: a power-of-two scaling)."""
    x = np.asarray(x, dtype=np.float32).astype(np.float64)
    return np.floor(x * float(FX_ONE)).astype(np.uint64)


def line_keys(mass: np.ndarray) -> np.ndarray:
    """mass[4, m] fp32 (vert or slash per probe group) -> uint64 ranking key per line."""
    return fx(mass).sum(axis=0, dtype=np.uint64)


def topk_desc(keys: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest keys; ties go to the lower index. Returned in selection order."""
    k = max(0, min(int(k), len(keys)))
    if keys.dtype.kind == "f":
        order = np.argsort(-keys, kind="stable")
    else:
        order = np.argsort(keys.max(initial=0) - keys, kind="stable")
    return order[:k]


# ----------------------------------------------------------------------------- index estimation
def build_vertical_slash(vert: np.ndarray, slash: np.ndarray, k_v: int, k_s: int, q1: int
                         ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """V = top-k_v columns of [0, q1); S = {0} + top-(k_s - 1) offsets of [1, q1); D from S."""
    kv = line_keys(vert[:, :q1])
    V = np.sort(topk_desc(kv, k_v)).astype(np.int32)
    ks = line_keys(slash[:, :q1])
    rest = topk_desc(ks[1:], max(0, min(k_s, q1) - 1)) + 1
    S = np.sort(np.concatenate([[0], rest])).astype(np.int32)
    nb = q1 // B
    deltas = np.unique(np.concatenate([S // B, (S + B - 1) // B]))
    D = deltas[deltas < nb].astype(np.int32)
    return V, S, D


def build_block_sparse(bscore: np.ndarray, k_b: int, qb_lo: int, qb_hi: int) -> List[np.ndarray]:
    """sel(qb) = {qb} + top-(min(k_b, qb+1) - 1) of bscore[qb - qb_lo, 0:qb], fp32 compare, ties -> lower kb."""
    out = []
    for qb in range(qb_lo, qb_hi):
        row = np.asarray(bscore[qb - qb_lo, :qb], dtype=np.float32)
        take = min(int(k_b), qb + 1) - 1
        sel = topk_desc(row, take)
        out.append(np.sort(np.concatenate([sel, [qb]])).astype(np.int32))
    return out


def build_indices(cand: Candidate, q0: int, q1: int, vert=None, slash=None, bscore=None) -> IndexSet:
    """Index set of one candidate on segment [q0, q1). bscore rows cover query blocks [q0/64, q1/64)."""
    ix = IndexSet(cand=cand, q0=q0, q1=q1)
    if cand.pattern == VERTICAL_SLASH:
        ix.V, ix.S, ix.D = build_vertical_slash(vert, slash, cand.b0, cand.b1, q1)
    elif cand.pattern == BLOCK_SPARSE:
        ix.blk = build_block_sparse(bscore, cand.b0, q0 // B, q1 // B)
    return ix


# ----------------------------------------------------------------------------- masks
def mask_rows(ix: IndexSet, rows: np.ndarray, n_keys: int) -> np.ndarray:
    """Boolean rows of the binary mask M (without the causal part) for keys [0, n_keys)."""
    c = ix.cand
    rows = np.asarray(rows)
    j = np.arange(n_keys)[None, :]
    i = rows[:, None]
    if c.pattern == DENSE:
        return np.ones((len(rows), n_keys), dtype=bool)
    if c.pattern == A_SHAPE:
        return (j < c.b0) | (i - j < c.b1)
    if c.pattern == VERTICAL_SLASH:
        col = np.zeros(n_keys, dtype=bool)
        col[ix.V[ix.V < n_keys]] = True
        if c.strict:
            off = np.zeros(max(n_keys, int(rows.max()) + 1, int(ix.S.max()) + 1) + 1, dtype=bool)
            off[ix.S] = True
            diff = i - j
            return col[None, :] | ((diff >= 0) & off[np.clip(diff, 0, len(off) - 1)])
        nb = max(max(n_keys, int(rows.max()) + 1) // B, int(ix.D.max())) + 2
        dl = np.zeros(nb, dtype=bool)
        dl[ix.D] = True
        delta = i // B - j // B
        return col[None, :] | ((delta >= 0) & dl[np.clip(delta, 0, nb - 1)])
    if c.pattern == BLOCK_SPARSE:
        M = np.zeros((len(rows), n_keys), dtype=bool)
        kb = np.arange(n_keys) // B
        for t, r in enumerate(rows):
            sel = ix.blk[int(r) // B - ix.q0 // B]
            M[t] = np.isin(kb, sel)
        return M
    raise ValueError("unknown pattern")


def explicit_mask(ix: IndexSet, n: int) -> np.ndarray:
    """Full n x n boolean mask including causality (rows outside the segment are all False). Small n only."""
    M = np.zeros((n, n), dtype=bool)
    rows = np.arange(ix.q0, ix.q1)
    M[rows] = mask_rows(ix, rows, n) & (np.arange(n)[None, :] <= rows[:, None])
    return M


# ----------------------------------------------------------------------------- pair counts (closed forms)
def pairs(ix: IndexSet) -> int:
    """Number of (i, j) with M[i, j] = 1 and j <= i over the segment's rows, in closed form."""
    c, q0, q1 = ix.cand, ix.q0, ix.q1
    if c.pattern == DENSE:
        return (q1 * (q1 + 1) - q0 * (q0 + 1)) // 2
    if c.pattern == A_SHAPE:
        cap = c.b0 + c.b1
        return int(sum(min(i + 1, cap) for i in range(q0, q1)))
    if c.pattern == BLOCK_SPARSE:
        return int(sum((len(sel) - 1) * B * B + B * (B + 1) // 2 for sel in ix.blk))
    if c.pattern == VERTICAL_SLASH:
        if c.strict:
            raise ValueError("closed form is defined for the executed BLOCK form")
        D = ix.D.astype(np.int64)
        has0 = bool((D == 0).any())
        total = 0
        Vs = ix.V.astype(np.int64)
        for qb in range(q0 // B, q1 // B):
            n_off = int(((D >= 1) & (D <= qb)).sum())
            total += B * B * n_off + (B * (B + 1) // 2 if has0 else 0)
            # vertical keys not already covered by a block diagonal of this query block
            dlt = qb - Vs // B
            free = (dlt >= 0) & ~np.isin(dlt, D)
            lo = np.maximum(qb * B, Vs[free])      # rows i >= j
            total += int(((qb + 1) * B - lo).sum())
        return int(total)
    raise ValueError("unknown pattern")


# ----------------------------------------------------------------------------- coverage
def coverage_plain(ix: IndexSet, P_rows: np.ndarray) -> np.ndarray:
    """Section 3.2: probe mass covered by the candidate's mask, per probe group, by the plain definition.

    P_rows[64, q1] holds the exact probe attention rows (rows q1-64 .. q1-1).  Returns float64[4].
    """
    q1 = ix.q1
    rows = np.arange(q1 - R_PROBE, q1)
    M = mask_rows(ix, rows, q1) & (np.arange(q1)[None, :] <= rows[:, None])
    per_row = (P_rows * M).sum(axis=1)
    return per_row.reshape(N_GROUPS, R_PROBE // N_GROUPS).mean(axis=1)


def coverage_fx(ix: IndexSet, vert: np.ndarray, slash: np.ndarray) -> np.ndarray:
    """Fixed-point coverage sums cov_fx[4] (uint64) from the probe's column and offset masses.

    All probe rows lie in the last query block qb* of the segment, so a block-granular mask is a
    set of key columns for them and its covered mass is a sum of vert entries; the A-shape mask is
    a set of columns plus a set of offsets.  m_hat_g = cov_fx[g] / (16 * 2^32).
    Dense is not computed here (its coverage is 1 by definition).
    """
    c, q1 = ix.cand, ix.q1
    fv = fx(vert[:, :q1])
    qb_star = q1 // B - 1
    if c.pattern == A_SHAPE:
        n_sink, w = c.b0, c.b1
        fs = fx(slash[:, :q1])
        if w >= q1:                              # window alone covers every causal key
            return fs.sum(axis=1, dtype=np.uint64)
        if q1 - R_PROBE - w + 1 < n_sink:
            raise ValueError("A-shape sink and window overlap on the probe rows: use coverage_plain")
        return fv[:, :n_sink].sum(axis=1, dtype=np.uint64) + fs[:, :w].sum(axis=1, dtype=np.uint64)
    if c.pattern == VERTICAL_SLASH:
        if c.strict:
            raise ValueError("STRICT coverage needs the probe rows: use coverage_plain")
        kb = np.arange(q1) // B
        in_band = np.isin(qb_star - kb, ix.D)
        cov = fv[:, in_band].sum(axis=1, dtype=np.uint64)
        extra = ix.V[~in_band[ix.V]]
        return cov + fv[:, extra].sum(axis=1, dtype=np.uint64)
    if c.pattern == BLOCK_SPARSE:
        sel = ix.blk[qb_star - ix.q0 // B]
        kb = np.arange(q1) // B
        return fv[:, np.isin(kb, sel)].sum(axis=1, dtype=np.uint64)
    raise ValueError("coverage_fx is not defined for this pattern")


def m_hat_from_fx(cov: np.ndarray) -> Tuple[float, float]:
    """(m_hat, u): mean coverage over the 64 probe rows and the spread max_g - min_g of group coverages."""
    cov = np.asarray(cov, dtype=np.uint64)
    m_hat = float(int(cov.sum(dtype=np.uint64))) / float(R_PROBE * FX_ONE)
    mg = [float(int(v)) / float((R_PROBE // N_GROUPS) * FX_ONE) for v in cov]
    return m_hat, max(mg) - min(mg)


def default_library() -> List[Candidate]:
    """13-candidate online library: four budgets per sparse family in increasing order, then dense."""
    lib = [Candidate(A_SHAPE, 128, w) for w in (1024, 2048, 4096, 8192)]
    lib += [Candidate(VERTICAL_SLASH, kv, ks) for kv, ks in ((500, 3048), (1000, 6096), (2000, 12192), (4000, 24384))]
    lib += [Candidate(BLOCK_SPARSE, kb) for kb in (50, 100, 200, 400)]
    lib += [Candidate(DENSE)]
    return lib


def mixture_coverage_fx(ix: IndexSet, a_row: np.ndarray, i: int, n_keys: int) -> int:
    """Coverage of mask row i under the pooled probe's block resolution (Section 3.2 mixture rows): the probability of
    every visible key block (a_row, float32, 64 keys per block) is split evenly over the block's visible keys, and the
    row collects floor(a * 2^32) * (selected visible keys) // (visible keys) per block.  Plain definition: the mask row
    itself is built and counted key by key."""
    m = mask_rows(ix, np.array([i]), n_keys)[0]
    m = m & (np.arange(n_keys) <= i)
    total = 0
    for kb in range(i // B + 1):
        lo, hi = kb * B, min(kb * B + B - 1, i)
        num = int(m[lo:hi + 1].sum())
        total += int(fx(np.float32(a_row[kb]))) * num // (hi - lo + 1)
    return total


def mixture_u(covmix: np.ndarray, rows_per_subset) -> float:
    """max_b m_b - min_b m_b with m_b = covmix[b] / (rows_b * 2^32) over the subsets in use."""
    ms = [float(int(covmix[b])) / (float(r) * float(FX_ONE)) for b, r in enumerate(rows_per_subset) if r > 0]
    return max(ms) - min(ms)
