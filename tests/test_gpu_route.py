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
    prm.reserved = int(kw.get("rescue_any", False))
    keep = []
    if kw.get("forced_dense"):
        fd = torch.zeros(cov.shape[0], dtype=torch.int32, device="cuda"); fd[list(kw["forced_dense"])] = 1
        prm.forced_dense = fd.data_ptr(); keep.append(fd)
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
