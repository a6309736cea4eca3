"""GPU parity: rs_route (single-block device solve) against the oracle, bit-exact decisions."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import c_library
from oracle import patterns as PT
from oracle import routing as RT

pytestmark = pytest.mark.gpu
C = PT.Candidate
LIB = PT.default_library()


def instance(rng, n_items, lib):
    cov = np.zeros((n_items, len(lib), 4), dtype=np.uint64)
    pairs = np.zeros((n_items, len(lib)), dtype=np.int64)
    for it in range(n_items):
        for c, cand in enumerate(lib):
            base = rng.uniform(0.3, 1.0) if cand.pattern != PT.DENSE else 1.0
            cov[it, c] = (np.clip(base + rng.uniform(-0.05, 0.05, 4), 0, 1) * 16 * 2 ** 32).astype(np.uint64)
            pairs[it, c] = rng.integers(1000, 100000) if cand.pattern != PT.DENSE else 200000
    return cov, pairs


def gpu_route(p, lib, cov, pairs, cost, vmax, **kw):
    stats = np.zeros((cov.shape[0], len(lib), 5), dtype=np.int64)
    stats[:, :, :4] = cov.astype(np.int64)
    stats[:, :, 4] = pairs
    prm = rs.rs_route_params()
    prm.budget = int(kw.get("budget", 0)); prm.t_probe = int(kw.get("t_probe", 0)); prm.alpha = kw.get("alpha", 1.0)
    prm.delta_q = kw.get("delta_q", 0.0)
    prm.use_cert = 0 if kw.get("cert_max") is None else 1
    prm.cert_max = 0.0 if kw.get("cert_max") is None else kw["cert_max"]
    prm.cert_mode = kw.get("cert_mode", rs.RS_CERT_REL); prm.expand_first = int(kw.get("expand_first", True))
    prm.rescue_any = int(kw.get("rescue_any", False))
    prm.backfill = int(kw.get("backfill", False))
    prm.global_pattern = int(kw.get("global_pattern", False))
    keep = []
    if kw.get("forced_dense"):
        fd = torch.zeros(cov.shape[0], dtype=torch.int32, device="cuda"); fd[list(kw["forced_dense"])] = 1
        prm.forced_dense = fd.data_ptr(); keep.append(fd)
    if kw.get("e") is not None:
        et = torch.from_numpy(np.ascontiguousarray(kw["e"], dtype=np.float64)).cuda()
        prm.e = et.data_ptr(); prm.beta = float(kw.get("beta", 0.0)); keep.append(et)
    if kw.get("fixed_choice") is not None:
        fc = torch.tensor(kw["fixed_choice"], dtype=torch.int32, device="cuda")
        prm.fixed_choice = fc.data_ptr(); keep.append(fc)
    choice = torch.full((cov.shape[0],), -1, dtype=torch.int32, device="cuda")
    rep = torch.zeros(24, dtype=torch.uint8, device="cuda")
    st = rs.new_status()
    cost_t = None if cost is None else torch.from_numpy(cost).cuda()
    rs.rs_route(p, c_library(lib), torch.from_numpy(stats).cuda(), cost_t, torch.from_numpy(vmax).cuda(), prm, choice, rep, st)
    r = rep.cpu().numpy()
    report = (int(r[:8].view(np.int64)[0]), float(r[8:16].view(np.float64)[0]), int(r[16:20].view(np.int32)[0]),
              int(r[20:24].view(np.int32)[0]))
    return choice.cpu().numpy(), report


@pytest.mark.parametrize("n_seg,Hq,Hkv", [(1, 32, 8), (4, 32, 8), (1, 4, 2)])
def test_route_is_bit_exact(n_seg, Hq, Hkv):
    rng = np.random.default_rng(n_seg * 100 + Hq)
    p = rs.Problem(Hq, Hkv, 64 * n_seg * 4, [64 * 4 * s for s in range(n_seg + 1)])
    n_items = n_seg * Hq
    for trial in range(6):
        cov, pairs = instance(rng, n_items, LIB)
        cost = 512 * pairs
        vmax_sg = rng.uniform(1, 14, (n_seg, Hkv)).astype(np.float32)
        vmax_item = np.array([vmax_sg[it // Hq, (it % Hq) // (Hq // Hkv)] for it in range(n_items)], np.float32)
        dense_total = int(cost[:, -1].sum())
        kw = dict(budget=int(dense_total * [0.05, 0.15, 0.4, 1.0, 0.001, 0.25][trial]), t_probe=12345,
                  alpha=[1.0, 0.5, 2.0, 1.0, 1.0, 0.0][trial],
                  cert_max=[None, 0.3, 0.05, 0.2, None, 2.0][trial],
                  cert_mode=[rs.RS_CERT_REL, rs.RS_CERT_REL, rs.RS_CERT_ABS, rs.RS_CERT_REL, 0, rs.RS_CERT_ABS][trial],
                  expand_first=trial != 3, delta_q=[0, 0.01, 0, 0, 0, 0.1][trial],
                  forced_dense=[0, n_items - 1] if trial == 1 else None, rescue_any=trial in (2, 5))
        use_cost = None if trial % 2 == 0 else cost
        got, rep = gpu_route(p, LIB, cov, pairs, use_cost, vmax_sg, **kw)
        want, wrep = RT.route(LIB, cov, cost, vmax_item, RT.RouteParams(
            budget=kw["budget"], t_probe=kw["t_probe"], alpha=kw["alpha"], delta_q=kw["delta_q"], cert_max=kw["cert_max"],
            cert_mode=kw["cert_mode"], expand_first=kw["expand_first"], forced_dense=kw["forced_dense"] or [],
            rescue_any=kw["rescue_any"]))
        assert np.array_equal(got, want), (trial, got, want)
        assert rep[0] == wrep.total_cost and rep[2] == wrep.n_fallback and rep[3] == wrep.feasible
        assert abs(rep[1] - wrep.total_risk) < 1e-9


def test_fixed_choice_and_ties():
    p = rs.Problem(4, 2, 256)
    lib = [C(PT.A_SHAPE, 8, 64), C(PT.DENSE)]
    cov = np.full((4, 2, 4), int(0.9 * 16 * 2 ** 32), dtype=np.uint64)
    pairs = np.array([[50, 100]] * 4, dtype=np.int64)
    got, rep = gpu_route(p, lib, cov, pairs, None, np.ones((1, 2), np.float32), budget=512 * 300)
    assert got.tolist() == [0, 0, 1, 1]              # equal ratios and savings: lower items move first
    got, rep = gpu_route(p, lib, cov, pairs, None, np.ones((1, 2), np.float32), budget=1, fixed_choice=[1, 0, 1, 0])
    assert got.tolist() == [1, 0, 1, 0] and rep[3] == 1
    got, rep = gpu_route(p, lib, cov, pairs, None, np.ones((1, 2), np.float32), budget=1)
    assert got.tolist() == [0, 0, 0, 0] and rep[3] == 0


def test_route_with_the_calibrated_predictor_is_bit_exact():
    """Eq. 4 with beta > 0: e comes from rs_regressor_eval (checked bit for bit against the oracle's predictor) and
    enters the risk; decisions and the reported risk are those of the oracle."""
    from oracle import calibration as CAL
    rng = np.random.default_rng(77)
    n_seg, Hq, Hkv = 2, 8, 2
    p = rs.Problem(Hq, Hkv, 1024, [0, 384, 1024])
    n_items = n_seg * Hq
    cov, pairs = instance(rng, n_items, LIB)
    for it in range(n_items):                     # pair counts below the segment's dense count, as real statistics are
        q0, q1 = p.seg_bounds[it // Hq], p.seg_bounds[it // Hq + 1]
        dense = (q1 * (q1 + 1) - q0 * (q0 + 1)) // 2
        pairs[it] = rng.integers(dense // 50, dense, len(LIB)); pairs[it, -1] = dense
    descr = rng.uniform(0, 1, (n_items, 4)).astype(np.float32)
    w = [1.0, 0.5, 0.25, 0.125, 0.3, 0.07]
    bp_z = np.array([0.05, 0.3, 0.55, 0.9, 1.4]); bp_e = np.array([0.0, 0.02, 0.1, 0.1, 0.6])
    stats = np.zeros((n_items, len(LIB), 5), dtype=np.int64)
    stats[:, :, :4] = cov.astype(np.int64); stats[:, :, 4] = pairs
    e_dev = torch.full((n_items, len(LIB)), -1.0, dtype=torch.float64, device="cuda")
    rs.rs_regressor_eval(p, c_library(LIB), torch.from_numpy(stats).cuda(), torch.from_numpy(descr).cuda(), w, bp_z, bp_e,
                         e_dev, rs.new_status())
    seg_of = [(p.seg_bounds[it // Hq], p.seg_bounds[it // Hq + 1]) for it in range(n_items)]
    e_want = CAL.regressor_eval(LIB, cov, pairs, descr, seg_of, w, bp_z, bp_e)
    assert np.array_equal(e_dev.cpu().numpy(), e_want)
    assert len(np.unique(e_want)) >= 3            # the instance exercises several steps of the table
    cost = 512 * pairs
    vmax_sg = rng.uniform(1, 4, (n_seg, Hkv)).astype(np.float32)
    vmax_item = np.array([vmax_sg[it // Hq, (it % Hq) // (Hq // Hkv)] for it in range(n_items)], np.float32)
    for beta, budget_frac in ((0.0, 0.2), (1.0, 0.2), (4.0, 0.1), (0.5, 0.5)):
        kw = dict(budget=int(cost[:, -1].sum() * budget_frac), t_probe=1000, alpha=1.0, cert_max=0.4, e=e_want, beta=beta)
        got, rep = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, **kw)
        want, wrep = RT.route(LIB, cov, cost, vmax_item, RT.RouteParams(budget=kw["budget"], t_probe=1000, alpha=1.0,
                                                                         cert_max=0.4, beta=beta, e=e_want))
        assert np.array_equal(got, want), beta
        assert rep[0] == wrep.total_cost and rep[1] == wrep.total_risk and rep[2] == wrep.n_fallback
    # the predictor changes decisions on this instance
    a, _ = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, budget=int(cost[:, -1].sum() * 0.2), alpha=1.0)
    b, _ = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, budget=int(cost[:, -1].sum() * 0.2), alpha=1.0, e=e_want, beta=4.0)
    assert not np.array_equal(a, b)


def test_output_error_rows():
    rng = np.random.default_rng(3)
    a = torch.from_numpy(rng.standard_normal((3, 70, 128)).astype(np.float32)).cuda()
    b = a + torch.from_numpy((0.01 * rng.standard_normal((3, 70, 128))).astype(np.float32)).cuda()
    for dt in (torch.float32, torch.bfloat16):
        x, y = a.to(dt), b.to(dt)
        err = torch.zeros(210, device="cuda"); nrm = torch.zeros(210, device="cuda")
        rs.rs_output_error(x, y, err, nrm, rs.new_status())
        xd, yd = x.double().cpu().numpy().reshape(210, 128), y.double().cpu().numpy().reshape(210, 128)
        assert np.allclose(err.cpu().numpy(), np.sqrt(((xd - yd) ** 2).sum(axis=1)), rtol=1e-5, atol=1e-7)
        assert np.allclose(nrm.cpu().numpy(), np.sqrt((xd ** 2).sum(axis=1)), rtol=1e-5)


def test_backfill_is_bit_exact_and_never_worse():
    rng = np.random.default_rng(5)
    p = rs.Problem(32, 8, 512)
    improved = 0
    for trial in range(6):
        cov, pairs = instance(rng, 32, LIB)
        cost = 512 * pairs
        vmax_sg = np.ones((1, 8), dtype=np.float32)
        budget = int(cost[:, -1].sum() * [0.1, 0.2, 0.3, 0.5, 0.05, 0.15][trial])
        base, brep = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, budget=budget, alpha=1.0)
        got, rep = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, budget=budget, alpha=1.0, backfill=True)
        want, wrep = RT.route(LIB, cov, cost, np.ones(32, np.float32), RT.RouteParams(budget=budget, backfill=True))
        assert np.array_equal(got, want) and rep[0] == wrep.total_cost and rep[1] == wrep.total_risk
        assert rep[0] <= budget and rep[1] <= brep[1] and rep[0] >= brep[0]
        improved += int(rep[1] < brep[1])
        # nothing that fits is left
        R, _ = RT.risks(LIB, cov, 1.0)
        for it in range(32):
            for k in range(len(LIB)):
                dT = int(cost[it, k]) - int(cost[it, got[it]])
                assert not (dT > 0 and rep[0] + dT <= budget and R[it, k] < R[it, got[it]])
    assert improved >= 1


def test_route_with_many_ties_and_non_monotone_sequences():
    """Coarsely quantised coverages and costs: many substitutions share a ratio, many items' sequences are not monotone;
    the device solve (sequences precomputed per item, merged by a sort of running maxima) must still take exactly the
    substitutions of the oracle's step-by-step greedy loop."""
    rng = np.random.default_rng(2024)
    for n_seg, Hq, Hkv in ((5, 32, 8), (1, 32, 8), (3, 8, 2)):
        p = rs.Problem(Hq, Hkv, 64 * n_seg * 2, [128 * s for s in range(n_seg + 1)])
        n_items = n_seg * Hq
        for trial in range(4):
            cov = np.zeros((n_items, len(LIB), 4), dtype=np.uint64)
            pairs = np.zeros((n_items, len(LIB)), dtype=np.int64)
            for it in range(n_items):
                for c, cand in enumerate(LIB):
                    lvl = rng.integers(2, 9) if cand.pattern != PT.DENSE else 8          # coverage in eighths
                    cov[it, c] = np.uint64(lvl * 2 * 2 ** 32)
                    pairs[it, c] = 1000 * rng.integers(1, 12) if cand.pattern != PT.DENSE else 20000
            cost = 512 * pairs
            vmax_sg = np.ones((n_seg, Hkv), dtype=np.float32)
            budget = int(cost[:, -1].sum() * [0.08, 0.2, 0.45, 0.02][trial])
            got, rep = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, budget=budget, alpha=1.0, backfill=trial == 2)
            want, wrep = RT.route(LIB, cov, cost, np.ones(n_items, np.float32), RT.RouteParams(budget=budget, backfill=trial == 2))
            assert np.array_equal(got, want), (n_seg, trial)
            assert rep[0] == wrep.total_cost and rep[1] == wrep.total_risk and rep[3] == wrep.feasible


@pytest.mark.parametrize("n_seg,Hq,Hkv", [(1, 32, 8), (4, 32, 8), (64, 32, 8)])
def test_layer_level_router_is_bit_exact(n_seg, Hq, Hkv):
    """One candidate for the whole layer: same decision, cost, risk (bit for bit) and fallback count as the oracle,
    on the shared-memory path and (2048 items) on the path that reads the tables from global memory."""
    rng = np.random.default_rng(900 + n_seg)
    p = rs.Problem(Hq, Hkv, 64 * n_seg * 2, [128 * s for s in range(n_seg + 1)])
    n_items = n_seg * Hq
    for trial in range(5):
        cov, pairs = instance(rng, n_items, LIB)
        cost = 512 * pairs
        vmax_sg = np.ones((n_seg, Hkv), dtype=np.float32)
        dense_total = int(cost[:, -1].sum())
        budget = int(dense_total * [0.05, 0.2, 0.5, 1.0, 0.0001][trial])
        cert_max = [None, 0.3, None, 0.3, None][trial]
        got, rep = gpu_route(p, LIB, cov, pairs, cost, vmax_sg, budget=budget, t_probe=77, global_pattern=True,
                             cert_max=cert_max)
        want, wrep = RT.route(LIB, cov, cost, np.ones(n_items, np.float32),
                              RT.RouteParams(budget=budget, t_probe=77, global_pattern=True, cert_max=cert_max))
        assert np.array_equal(got, want)
        assert rep == (wrep.total_cost, wrep.total_risk, wrep.n_fallback, wrep.feasible)
        if cert_max is None:
            assert len(set(got.tolist())) == 1
