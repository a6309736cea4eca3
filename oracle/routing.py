"""Oracle: risk score (Eq. 4), latency-constrained routing (Eq. 6-8) and the fallback rule (Section 3.4).

Test infrastructure only; never imported by the product path.

Items are (segment, head) pairs; every item picks exactly one candidate of the library (Eq. 7) and the
summed cost plus the probe cost must not exceed the layer budget T (Eq. 8).  The paper solves this with
a greedy heuristic: start from the zero-risk dense choice everywhere and repeatedly apply the
substitution with the best risk increase per unit of cost saved until the budget is met.  Then items
whose lower-confidence mass is too small first take a larger budget of the same family and finally
dense.  The paper names no tie-break and no order of the fallback walk; the order used here is this
build's reading (parity unpinned beyond the invariants the tests check).

Arithmetic: coverage arrives as exact fixed-point integers, costs are integers (FLOPs or nanoseconds),
so totals are exact; risks are IEEE doubles computed as (1 - m_hat) + alpha * u with each operation
rounded separately; a substitution's ratio is the single IEEE division dR / dT, and substitutions are
ordered by the tuple (ratio, larger saving first, lower item, lower candidate), a total order, so the
chosen substitution does not depend on the order in which candidates are examined.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from itertools import product
from typing import List, Optional, Sequence

import numpy as np

from .patterns import DENSE, Candidate, m_hat_from_fx

CERT_ABS, CERT_REL = 0, 1


@dataclass
class RouteParams:
    budget: int                      # T_l, same integer unit as cost
    t_probe: int = 0
    alpha: float = 1.0               # weight of the probe-subset disagreement u
    beta: float = 0.0                # weight of the calibrated error predictor e (0: training-free router)
    e: Optional[np.ndarray] = None   # [items, n_cand] float64 predictor values (calibration.regressor_eval)
    delta_q: float = 0.0             # one-sided residual quantile: m_low = max(0, m_hat - delta_q)
    cert_max: Optional[float] = None  # fallback fires while certificate > cert_max (None: no fallback)
    cert_mode: int = CERT_REL        # REL: 2(1 - m_low);  ABS: 2(1 - m_low) * vmax
    expand_first: bool = True        # try the next larger budget of the family before dense
    rescue_any: bool = False         # before dense, take the cheapest sparse candidate of any family that passes
    backfill: bool = False           # spend leftover budget on the best risk decrease per added cost (before fallback)
    u_mix: Optional[np.ndarray] = None   # [items, n_cand] disagreement among the mixture's row subsets (replaces u)
    global_pattern: bool = False     # comparison router of Section 4: one candidate for the whole layer
    forced_dense: Sequence[int] = field(default_factory=list)   # items forced to dense last
    fixed_choice: Optional[Sequence[int]] = None                 # bypasses the solve and the fallback


@dataclass
class RouteReport:
    total_cost: int
    total_risk: float
    n_fallback: int
    feasible: int


def risks(lib: List[Candidate], cov_fx: np.ndarray, alpha: float, beta: float = 0.0, e: Optional[np.ndarray] = None,
          u_mix: Optional[np.ndarray] = None):
    """R[item][c] = (1 - m_hat) + alpha * u + beta * e (Eq. 4); dense has m_hat = 1, u = 0, e = 0, R = 0."""
    n_items, n_cand = cov_fx.shape[0], len(lib)
    R = np.zeros((n_items, n_cand), dtype=np.float64)
    M = np.ones((n_items, n_cand), dtype=np.float64)
    for it in range(n_items):
        for c, cand in enumerate(lib):
            if cand.pattern == DENSE:
                continue
            m_hat, u = m_hat_from_fx(cov_fx[it, c])
            if u_mix is not None:
                u = float(u_mix[it, c])
            M[it, c] = m_hat
            R[it, c] = (1.0 - m_hat) + alpha * u
            if e is not None and beta != 0.0:
                R[it, c] = R[it, c] + beta * float(e[it, c])
    return R, M


def _dense_index(lib: List[Candidate]) -> int:
    for c, cand in enumerate(lib):
        if cand.pattern == DENSE:
            return c
    raise ValueError("the library must contain the dense candidate")


def greedy_solve(R: np.ndarray, cost: np.ndarray, dense_c: int, budget: int, t_probe: int):
    """Greedy substitution for Eq. 6-8. Returns (choice, total, feasible)."""
    n_items, n_cand = R.shape
    choice = [dense_c] * n_items
    total = int(t_probe) + sum(int(cost[it, dense_c]) for it in range(n_items))
    feasible = 1
    while total > budget:
        best = None                                   # (ratio, -dT, item, cand): smallest tuple wins
        for it in range(n_items):
            cur = choice[it]
            for k in range(n_cand):
                dT = int(cost[it, cur]) - int(cost[it, k])
                if dT <= 0:
                    continue
                dR = float(R[it, k]) - float(R[it, cur])
                key = (dR / float(dT), -dT, it, k)    # one IEEE division; ties: larger saving, lower item, lower k
                if best is None or key < best:
                    best = key
        if best is None:
            feasible = 0
            break
        _, neg_dT, it, k = best
        choice[it] = k
        total += neg_dT
    return choice, total, feasible


def global_solve(R: np.ndarray, cost: np.ndarray, budget: int, t_probe: int):
    """The layer-level router the paper compares against (Section 4, baselines): Eq. 6-8 with the extra constraint that
    every item takes the same candidate.  Among the candidates whose summed cost meets the budget the one with the
    smallest summed risk wins (ties: cheaper, lower index); if none does, the cheapest one is taken and the result is
    marked infeasible.  Risks are summed in item order, one rounding per addition."""
    n_items, n_cand = R.shape
    best = None                                       # (infeasible, risk or 0, cost, c)
    for c in range(n_cand):
        tot = int(t_probe) + sum(int(cost[it, c]) for it in range(n_items))
        risk = 0.0
        for it in range(n_items):
            risk += float(R[it, c])
        key = (0, risk, tot, c) if tot <= budget else (1, 0.0, tot, c)
        if best is None or key < best:
            best = key
    infeasible, _, tot, c = best
    return [c] * n_items, tot, 1 - infeasible


def backfill(choice: List[int], total: int, R: np.ndarray, cost: np.ndarray, budget: int):
    """Greedy back-fill: while some substitution to a more expensive, less risky candidate still fits the budget, apply
    the one with the largest risk decrease per unit of added cost (ties: cheaper, lower item, lower candidate).
    The paper does not describe this pass; it is this build's extension of the greedy heuristic."""
    n_items, n_cand = R.shape
    while True:
        best = None
        for it in range(n_items):
            cur = choice[it]
            for k in range(n_cand):
                dT = int(cost[it, k]) - int(cost[it, cur])
                if dT <= 0 or total + dT > budget:
                    continue
                dR = float(R[it, k]) - float(R[it, cur])
                if not dR < 0.0:
                    continue
                key = (dR / float(dT), dT, it, k)
                if best is None or key < best:
                    best = key
        if best is None:
            return choice, total
        _, dT, it, k = best
        choice[it] = k
        total += dT


def _next_larger(lib: List[Candidate], c: int) -> Optional[int]:
    """Index of the next entry of the same family after c (library lists a family by increasing budget)."""
    for k in range(c + 1, len(lib)):
        if lib[k].pattern == lib[c].pattern:
            return k
    return None


def route(lib: List[Candidate], cov_fx: np.ndarray, cost: np.ndarray, vmax: np.ndarray, p: RouteParams):
    """Full routing of one layer. cov_fx[items, n_cand, 4] uint64, cost[items, n_cand] int64, vmax[items] fp32."""
    n_items = cov_fx.shape[0]
    dense_c = _dense_index(lib)
    R, M = risks(lib, cov_fx, p.alpha, p.beta, p.e, p.u_mix)
    n_fallback = 0
    if p.fixed_choice is not None:
        choice = [int(c) for c in p.fixed_choice]
        feasible = 1
    else:
        if p.global_pattern:
            choice, total, feasible = global_solve(R, cost, int(p.budget), int(p.t_probe))
        else:
            choice, total, feasible = greedy_solve(R, cost, dense_c, int(p.budget), int(p.t_probe))
        if p.backfill and feasible and not p.global_pattern:
            choice, total = backfill(choice, total, R, cost, int(p.budget))
        if p.cert_max is not None:
            for it in range(n_items):
                fired = False
                while lib[choice[it]].pattern != DENSE:
                    m_low = max(0.0, float(M[it, choice[it]]) - p.delta_q)
                    cert = 2.0 * (1.0 - m_low)
                    if p.cert_mode == CERT_ABS:
                        cert = cert * float(np.float32(vmax[it]))
                    if not cert > p.cert_max:
                        break
                    fired = True
                    nxt = _next_larger(lib, choice[it]) if p.expand_first else None
                    if nxt is None and p.rescue_any:
                        # "switches to dense attention if no sparse candidate satisfies the threshold": look at every
                        # sparse candidate, keep those whose certificate passes, take the cheapest (ties: lower index)
                        best = None
                        for k, cand in enumerate(lib):
                            if cand.pattern == DENSE:
                                continue
                            ck = 2.0 * (1.0 - max(0.0, float(M[it, k]) - p.delta_q))
                            if p.cert_mode == CERT_ABS:
                                ck = ck * float(np.float32(vmax[it]))
                            if not ck > p.cert_max and (best is None or int(cost[it, k]) < int(cost[it, best])):
                                best = k
                        nxt = best
                    choice[it] = nxt if nxt is not None else dense_c
                n_fallback += int(fired)
    for it in p.forced_dense:
        choice[int(it)] = dense_c
    total = int(p.t_probe) + sum(int(cost[it, choice[it]]) for it in range(n_items))
    risk = 0.0
    for it in range(n_items):
        risk += float(R[it, choice[it]])
    return np.asarray(choice, dtype=np.int32), RouteReport(total, risk, n_fallback, feasible)


def exhaustive_optimum(R: np.ndarray, cost: np.ndarray, budget: int, t_probe: int):
    """Exact multiple-choice knapsack by enumeration (tiny instances only). Returns (risk, choice) or None."""
    n_items, n_cand = R.shape
    best = None
    for combo in product(range(n_cand), repeat=n_items):
        tot = int(t_probe) + sum(int(cost[i, c]) for i, c in enumerate(combo))
        if tot > budget:
            continue
        r = sum(float(R[i, c]) for i, c in enumerate(combo))
        if best is None or r < best[0]:
            best = (r, combo)
    return best
