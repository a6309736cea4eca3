"""Pins for the oracle's risk (Eq. 4), routing (Eq. 6-8) and fallback (Section 3.4). CPU only."""
import numpy as np
import pytest

from oracle import patterns as PT
from oracle import routing as RT

C = PT.Candidate
LIB = [C(PT.A_SHAPE, 8, 64), C(PT.A_SHAPE, 8, 128), C(PT.VERTICAL_SLASH, 8, 8), C(PT.BLOCK_SPARSE, 2), C(PT.DENSE)]
DENSE_C = 4


def _instance(rng, n_items=4):
    cov = np.zeros((n_items, len(LIB), 4), dtype=np.uint64)
    cost = np.zeros((n_items, len(LIB)), dtype=np.int64)
    for it in range(n_items):
        for c in range(len(LIB) - 1):
            base = rng.uniform(0.2, 1.0)
            cov[it, c] = (np.clip(base + rng.uniform(-0.1, 0.1, 4), 0, 1) * 16 * 2 ** 32).astype(np.uint64)
            cost[it, c] = rng.integers(10, 90)
        cov[it, 1] = np.maximum(cov[it, 1], cov[it, 0])      # larger budget of a family covers at least as much
        cost[it, 1] = max(cost[it, 1], cost[it, 0] + 1)
        cost[it, DENSE_C] = 100
    return cov, cost


def test_risk_formula():
    cov = np.zeros((1, len(LIB), 4), dtype=np.uint64)
    cov[0, 0] = np.array([0.5, 0.75, 1.0, 0.25]) * 16 * 2 ** 32
    R, M = RT.risks(LIB, cov, alpha=2.0)
    assert M[0, 0] == 0.625 and R[0, 0] == (1 - 0.625) + 2.0 * 0.75
    assert R[0, DENSE_C] == 0.0 and M[0, DENSE_C] == 1.0


def test_constraints_and_bound_against_exhaustive_optimum():
    rng = np.random.default_rng(0)
    n_opt = 0
    for trial in range(60):
        cov, cost = _instance(rng)
        budget = int(rng.integers(30, 420))
        choice, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=budget, t_probe=5))
        assert choice.shape == (4,) and np.all((choice >= 0) & (choice < len(LIB)))      # Eq. 7
        R, _ = RT.risks(LIB, cov, 1.0)
        best = RT.exhaustive_optimum(R, cost, budget, 5)
        if best is None:
            assert rep.feasible == 0
            assert all(cost[i, choice[i]] == cost[i].min() for i in range(4))
        else:
            assert rep.feasible == 1 and rep.total_cost <= budget                          # Eq. 8
            assert rep.total_risk >= best[0] - 1e-12
            n_opt += abs(rep.total_risk - best[0]) < 1e-12
        assert rep.total_cost == 5 + sum(cost[i, choice[i]] for i in range(4))
    assert n_opt > 5          # the heuristic does find the optimum on a fair share of instances


def test_trivial_budgets():
    rng = np.random.default_rng(1)
    cov, cost = _instance(rng)
    choice, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=405, t_probe=5))
    assert np.all(choice == DENSE_C) and rep.total_risk == 0.0 and rep.feasible == 1
    choice, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=1, t_probe=5))
    assert rep.feasible == 0


def test_greedy_takes_best_ratio_first():
    lib = [C(PT.A_SHAPE, 8, 64), C(PT.DENSE)]
    cov = np.zeros((2, 2, 4), dtype=np.uint64)
    cov[0, 0] = np.uint64(int(0.9 * 16 * 2 ** 32))      # item 0 loses 0.1 mass for 50 units
    cov[1, 0] = np.uint64(int(0.5 * 16 * 2 ** 32))      # item 1 loses 0.5 mass for 50 units
    cost = np.array([[50, 100], [50, 100]], dtype=np.int64)
    choice, rep = RT.route(lib, cov, cost, np.ones(2, np.float32), RT.RouteParams(budget=150))
    assert choice.tolist() == [0, 1]
    # equal ratios: the larger saving wins, then the lower item
    cov[1, 0] = cov[0, 0]
    choice, _ = RT.route(lib, cov, cost, np.ones(2, np.float32), RT.RouteParams(budget=150))
    assert choice.tolist() == [0, 1]


def test_fallback_expands_then_goes_dense_and_never_lowers_coverage():
    rng = np.random.default_rng(2)
    for trial in range(30):
        cov, cost = _instance(rng)
        base, _ = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=200))
        fb, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32),
                           RT.RouteParams(budget=200, cert_max=0.3, cert_mode=RT.CERT_REL))
        _, M = RT.risks(LIB, cov, 1.0)
        for it in range(4):
            assert M[it, fb[it]] >= M[it, base[it]]
            assert LIB[fb[it]].pattern == PT.DENSE or 2 * (1 - M[it, fb[it]]) <= 0.3
            if fb[it] != base[it]:
                assert LIB[fb[it]].pattern in (PT.DENSE, LIB[base[it]].pattern)
        assert rep.n_fallback == int((fb != base).sum())
        direct, _ = RT.route(LIB, cov, cost, np.ones(4, np.float32),
                             RT.RouteParams(budget=200, cert_max=0.3, expand_first=False))
        assert all(direct[it] in (base[it], DENSE_C) for it in range(4))


def test_abs_mode_scales_with_vmax_and_delta_q_shifts():
    cov = np.zeros((1, len(LIB), 4), dtype=np.uint64)
    cov[0, :4] = np.uint64(int(0.99 * 16 * 2 ** 32))
    cost = np.array([[10, 20, 30, 40, 100]], dtype=np.int64)
    p = dict(budget=50, cert_max=0.05)
    assert RT.route(LIB, cov, cost, np.float32([1.0]), RT.RouteParams(cert_mode=RT.CERT_ABS, **p))[0][0] != DENSE_C
    assert RT.route(LIB, cov, cost, np.float32([13.5]), RT.RouteParams(cert_mode=RT.CERT_ABS, **p))[0][0] == DENSE_C
    assert RT.route(LIB, cov, cost, np.float32([1.0]), RT.RouteParams(delta_q=0.02, **p))[0][0] == DENSE_C


def test_forced_dense_and_fixed_choice():
    rng = np.random.default_rng(3)
    cov, cost = _instance(rng)
    choice, _ = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=150, forced_dense=[1, 3]))
    assert choice[1] == DENSE_C and choice[3] == DENSE_C
    choice, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=1, fixed_choice=[0, 1, 2, 3]))
    assert choice.tolist() == [0, 1, 2, 3] and rep.n_fallback == 0


def test_rescue_takes_the_cheapest_passing_candidate_of_any_family():
    cov = np.zeros((1, len(LIB), 4), dtype=np.uint64)
    for c, m in enumerate([0.5, 0.6, 0.99, 0.995]):          # A-shape candidates fail, VS and BS pass
        cov[0, c] = np.uint64(int(m * 16 * 2 ** 32))
    cost = np.array([[10, 20, 60, 50, 100]], dtype=np.int64)
    base = RT.RouteParams(budget=15, cert_max=0.05)
    assert RT.route(LIB, cov, cost, np.float32([1.0]), base)[0].tolist() == [DENSE_C]
    rescued = RT.RouteParams(budget=15, cert_max=0.05, rescue_any=True)
    assert RT.route(LIB, cov, cost, np.float32([1.0]), rescued)[0].tolist() == [3]     # block-sparse is cheaper than VS
    cov[0, 2:4] = np.uint64(int(0.9 * 16 * 2 ** 32))
    assert RT.route(LIB, cov, cost, np.float32([1.0]), rescued)[0].tolist() == [DENSE_C]


def test_backfill_uses_leftover_budget_without_exceeding_it():
    from oracle.routing import RouteParams, backfill, greedy_solve, risks, route
    rng = np.random.default_rng(12)
    lib = PT.default_library()
    for trial in range(5):
        n_items = 6
        cov = np.zeros((n_items, len(lib), 4), dtype=np.uint64)
        cost = np.zeros((n_items, len(lib)), dtype=np.int64)
        for it in range(n_items):
            for c, cand in enumerate(lib):
                base = rng.uniform(0.3, 1.0) if cand.pattern != PT.DENSE else 1.0
                cov[it, c] = np.full(4, int(base * 16 * 2 ** 32), dtype=np.uint64)
                cost[it, c] = rng.integers(100, 5000) if cand.pattern != PT.DENSE else 10000
        budget = int(cost[:, -1].sum() * 0.3)
        R, _ = risks(lib, cov, 1.0)
        ch, total, feas = greedy_solve(R, cost, len(lib) - 1, budget, 0)
        r0 = sum(R[i, ch[i]] for i in range(n_items))
        ch2, total2 = backfill(list(ch), total, R, cost, budget)
        r1 = sum(R[i, ch2[i]] for i in range(n_items))
        assert total2 <= budget and total2 >= total and r1 <= r0
        assert total2 == sum(int(cost[i, ch2[i]]) for i in range(n_items))
        for i in range(n_items):                                   # nothing that fits and lowers the risk is left
            for k in range(len(lib)):
                dT = int(cost[i, k]) - int(cost[i, ch2[i]])
                assert not (dT > 0 and total2 + dT <= budget and R[i, k] < R[i, ch2[i]])
        got, rep = route(lib, cov, cost, np.ones(n_items, np.float32), RouteParams(budget=budget, backfill=True))
        assert list(got) == ch2 and rep.total_cost == total2


def test_greedy_order_is_the_order_of_running_maxima():
    """The step-by-step greedy loop takes the substitutions in the order obtained by sorting every item's own sequence
    entries by the running maximum of their keys (entries of one item by position): an entry whose key is smaller than
    an earlier key of its sequence is taken right after that earlier entry.  (The device solve relies on this.)"""
    from oracle.routing import greedy_solve, risks
    rng = np.random.default_rng(77)
    lib = PT.default_library()
    dense_c = len(lib) - 1
    for trial in range(8):
        n_items = 9
        cov = np.zeros((n_items, len(lib), 4), dtype=np.uint64)
        cost = np.zeros((n_items, len(lib)), dtype=np.int64)
        for it in range(n_items):
            for c, cand in enumerate(lib):
                lvl = rng.integers(2, 9) if cand.pattern != PT.DENSE else 8
                cov[it, c] = np.uint64(lvl * 2 * 2 ** 32)
                cost[it, c] = 1000 * rng.integers(1, 12) if cand.pattern != PT.DENSE else 20000
        R, _ = risks(lib, cov, 1.0)
        # every item's sequence from dense, key = (ratio, -dT, item, k)
        entries = []
        for it in range(n_items):
            cur, seq = dense_c, []
            while True:
                best = None
                for k in range(len(lib)):
                    dT = int(cost[it, cur]) - int(cost[it, k])
                    if dT <= 0:
                        continue
                    key = ((float(R[it, k]) - float(R[it, cur])) / float(dT), -dT, it, k)
                    if best is None or key < best:
                        best = key
                if best is None:
                    break
                seq.append(best)
                cur = best[3]
            run = None
            for j, key in enumerate(seq):
                run = key if run is None or key > run else run
                entries.append((run, j, key))
        order = [e[2] for e in sorted(entries, key=lambda e: (e[0], e[1]))]
        for frac in (0.05, 0.2, 0.5):
            budget = int(cost[:, dense_c].sum() * frac)
            choice, total, feas = greedy_solve(R, cost, dense_c, budget, 0)
            ch2, tot2 = [dense_c] * n_items, int(cost[:, dense_c].sum())
            for key in order:
                if tot2 <= budget:
                    break
                ch2[key[2]] = key[3]
                tot2 += key[1]
            assert ch2 == choice and tot2 == total, (trial, frac)


def test_global_router_is_the_best_constant_assignment():
    """One candidate for the whole layer (the layer-level comparison router of Section 4): the exhaustive optimum over
    the constant assignments, never better than the exhaustive optimum over all assignments."""
    rng = np.random.default_rng(7)
    n_feasible = 0
    for trial in range(60):
        cov, cost = _instance(rng)
        budget = int(rng.integers(60, 420))
        choice, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32),
                               RT.RouteParams(budget=budget, t_probe=5, global_pattern=True))
        assert len(set(choice.tolist())) == 1
        R, _ = RT.risks(LIB, cov, 1.0)
        constant = [(sum(R[i, c] for i in range(4)), 5 + int(cost[:, c].sum()), c) for c in range(len(LIB))
                    if 5 + int(cost[:, c].sum()) <= budget]
        if not constant:
            assert rep.feasible == 0 and int(cost[:, choice[0]].sum()) == min(int(cost[:, c].sum()) for c in range(len(LIB)))
            continue
        n_feasible += 1
        assert rep.feasible == 1 and rep.total_cost <= budget
        assert choice[0] == min(constant)[2]
        best = RT.exhaustive_optimum(R, cost, budget, 5)
        assert rep.total_risk >= best[0] - 1e-12
    assert n_feasible > 20
    # dense fits: the layer stays dense; nothing fits: cheapest candidate, marked infeasible
    cov, cost = _instance(rng)
    choice, rep = RT.route(LIB, cov, cost, np.ones(4, np.float32), RT.RouteParams(budget=405, t_probe=5, global_pattern=True))
    assert np.all(choice == DENSE_C) and rep.total_risk == 0.0


def _greedy_by_cross_multiplication(Rnum, den, cost, dense_c, budget, t_probe):
    """The greedy substitution with "risk per unit of cost" (Section 3.4: the risk-per-microsecond substitution) compared
    exactly: risks are the rationals Rnum / den, and dR1 / dT1 < dR2 / dT2 is decided as dR1 * dT2 < dR2 * dT1 in
    integers (dT > 0).  Ties: larger saving, lower item, lower candidate."""
    n_items, n_cand = Rnum.shape
    choice = [dense_c] * n_items
    total = t_probe + int(cost[:, dense_c].sum())
    while total > budget:
        best = None                     # (dR numerator, dT, item, k)
        for it in range(n_items):
            cur = choice[it]
            for k in range(n_cand):
                dT = int(cost[it, cur]) - int(cost[it, k])
                if dT <= 0:
                    continue
                dR = int(Rnum[it, k]) - int(Rnum[it, cur])
                if best is None:
                    best = (dR, dT, it, k)
                    continue
                lhs, rhs = dR * best[1], best[0] * dT          # dR / dT  vs  best dR / best dT
                if lhs < rhs or (lhs == rhs and (-dT, it, k) < (-best[1], best[2], best[3])):
                    best = (dR, dT, it, k)
        if best is None:
            return choice, total, 0
        choice[best[2]] = best[3]
        total -= best[1]
    return choice, total, 1


def test_one_division_orders_substitutions_like_exact_cross_multiplication():
    """The oracle ranks substitutions by the single IEEE division dR / dT inside the tuple (ratio, -dT, item, k).  The
    sentence it reads (Section 3.4, "greedily apply the risk-per-microsecond substitution") fixes the exact quotient;
    here the two are shown to agree wherever the quotient is decided exactly: risks that are multiples of 1/64 and
    integer costs below 2^20 make dR and dT exact, equal rationals divide to the same double and different rationals
    (which differ by more than 2^-46 relative) to different doubles.  Thousands of random instances with many exact ties
    between different (dR, dT) pairs -- 1/64 over 1 against 2/64 over 2 -- plus planted duplicates of whole items."""
    rng = np.random.default_rng(2608)
    n_cand, dense_c = 6, 5
    n_ties = 0
    for trial in range(3000):
        n_items = int(rng.integers(2, 7))
        Rnum = rng.integers(0, 40, size=(n_items, n_cand))           # risk = Rnum / 64
        cost = rng.integers(1, 24, size=(n_items, n_cand)) * int(rng.choice([1, 1000, 65536]))
        Rnum[:, dense_c] = 0
        cost[:, dense_c] = cost.max() + int(rng.integers(1, 9))
        if trial % 3 == 0 and n_items >= 3:                          # planted ties: an item repeated
            Rnum[2], cost[2] = Rnum[0], cost[0]
        R = Rnum.astype(np.float64) / 64.0
        budget = int(cost[:, dense_c].sum() * rng.uniform(0.05, 0.9))
        want = _greedy_by_cross_multiplication(Rnum, 64, cost, dense_c, budget, 3)
        got = RT.greedy_solve(R, cost, dense_c, budget, 3)
        assert (list(got[0]), got[1], got[2]) == (want[0], want[1], want[2]), trial
        # count instances where the first step already has an exact tie of the quotient between different pairs
        first = sorted((Rnum[it, k] * 1.0 / (cost[it, dense_c] - cost[it, k]), it, k)
                       for it in range(n_items) for k in range(n_cand - 1))
        n_ties += first[0][0] == first[1][0]
    assert n_ties > 100                                              # the tie-break branch really is exercised
