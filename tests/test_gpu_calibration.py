"""GPU: the offline calibration pass (Section 3.5) end to end on small seeded layers, its host statistics against the
oracle's restatement, and the calibrated router (Eq. 4 with beta > 0) against the oracle."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from paper_2608_29058_b200 import calibrate as CALIB
from gpu_helpers import dev_bf16, f64_heads
from oracle import attention as OA
from oracle import calibration as OCAL
from oracle import patterns as PT
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu

LIB = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_A_SHAPE, 64, 256), (rs.RS_VERTICAL_SLASH, 32, 96), (rs.RS_VERTICAL_SLASH, 64, 192),
       (rs.RS_BLOCK_SPARSE, 3, 0), (rs.RS_DENSE, 0, 0)]


def layer_inputs(seed, n=1024, Hq=4, Hkv=2):
    L = make_layer(tiny_spec(seed, n, Hq, Hkv))
    return L, dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"]), rs.Problem(Hq, Hkv, n)


def test_audit_records_match_the_oracle():
    L, Q, K, V, p = layer_inputs(11)
    recs = CALIB.audit_layer(Q, K, V, p, LIB, g=16)
    assert len(recs) == p.n_items * 5
    Qs, Ks, Vs = f64_heads(L)
    n = p.n_keys
    rows = np.arange(n)
    for h in (0, 3):
        O_d, lse_d = OA.dense_attention(Qs[h], Ks[h // 2], Vs[h // 2], rows)[:2]
        # candidate 1 = A-shape(64, 256): its mask is arithmetic, so the oracle needs nothing from the probe
        ix = PT.build_indices(PT.Candidate(PT.A_SHAPE, 64, 256), 0, n, None, None, None)
        O_s, lse_s, _ = OA.masked_attention(Qs[h], Ks[h // 2], Vs[h // 2], lambda rr, nk, ix=ix: PT.mask_rows(ix, rr, nk), rows)
        r = [x for x in recs if x["item"] == h and x["cand"] == 1][0]
        assert abs(r["m_true"] - OCAL.true_mass(lse_s, lse_d)) < 2e-3
        want_err = np.sqrt(((O_d.astype(np.float64) - O_s.astype(np.float64)) ** 2).sum(axis=1)).mean()
        # both GPU outputs are rounded to bf16: their difference carries up to 2^-8 of the output norm per operand
        noise = 2.0 ** -7 * np.sqrt((O_d.astype(np.float64) ** 2).sum(axis=1)).mean()
        assert abs(r["mean_err"] - want_err) < 0.02 * want_err + noise
        assert r["row_coverage"] == 1.0                              # Eq. 5 with the exact mass holds on every row
        assert 0.0 <= r["m_hat"] <= 1.0 and 0.0 <= r["u"] <= 1.0


def test_calibration_statistics_match_the_oracle_and_cover():
    recs, held = [], []
    for seed in (21, 22):
        _, Q, K, V, p = layer_inputs(seed)
        recs += CALIB.audit_layer(Q, K, V, p, LIB, g=16)
    _, Q, K, V, p = layer_inputs(23)
    held = CALIB.audit_layer(Q, K, V, p, LIB, g=16)
    out = CALIB.calibrate(recs, {"other_seed": held}, q=0.9, g=16)
    res = [r["m_hat"] - r["m_true"] for r in recs]
    assert out["delta_q"] == OCAL.one_sided_quantile(res, 0.9)
    assert out["coverage_in_domain"]["mass"] >= 0.9
    assert out["coverage_in_domain"]["certificate"] >= out["coverage_without_delta"]["certificate"]
    assert 0.0 <= out["coverage_held_out_other_seed"]["mass"] <= 1.0
    reg = out["regressor"]
    assert all(w >= 0 for w in reg["w"]) and len(reg["bp_z"]) <= 64
    assert np.all(np.diff(reg["bp_z"]) > 0) and np.all(np.diff(reg["bp_e"]) >= 0)
    # the step function is the isotonic fit of the oracle on the same projections
    X = np.array([r["features"] for r in recs]); y = np.array([r["mean_err"] / r["vmax"] for r in recs])
    bz, be = OCAL.isotonic_fit(X @ np.array(reg["w"]), y)
    if len(bz) <= 64:
        assert np.allclose(bz, reg["bp_z"]) and np.allclose(be, reg["bp_e"])
    assert reg["fit_rmse"] <= reg["target_std"] + 1e-12             # never worse than predicting the mean... of a monotone fit


def test_calibrated_router_matches_the_oracle():
    from oracle import routing as RT
    L, Q, K, V, p = layer_inputs(31)
    _, Q2, K2, V2, _ = layer_inputs(32)
    calib = CALIB.calibrate(CALIB.audit_layer(Q2, K2, V2, p, LIB, g=16), q=0.9, g=16)
    layer = rs.RoutedPrefillLayer(p, LIB, rs.RouteConfig(budget_frac=0.35, cert_max=0.5, beta=2.0))
    layer.use_calibration(calib)
    layer.forward(Q, K, V)
    rs.check_status(layer.status, "calibrated layer")
    got = layer.choice.cpu().numpy()
    stats = layer.stats.cpu().numpy()
    cov = stats[:, :, :4].astype(np.uint64); pairs = stats[:, :, 4]
    descr = layer.pp["descr"].reshape(p.n_items, 4).cpu().numpy()
    lib = [PT.Candidate(*c) if c[0] != rs.RS_BLOCK_SPARSE else PT.Candidate(c[0], c[1]) for c in LIB]
    reg = calib["regressor"]
    e = OCAL.regressor_eval(lib, cov, pairs, descr, [(0, p.n_keys)] * p.n_items, reg["w"], np.array(reg["bp_z"]), np.array(reg["bp_e"]))
    assert np.array_equal(layer.e_risk.cpu().numpy(), e)
    vmax = layer.vmax.cpu().numpy()
    vmax_item = np.array([vmax[0, h // 2] for h in range(p.n_items)], np.float32)
    want, _ = RT.route(lib, cov, 512 * pairs, vmax_item, RT.RouteParams(
        budget=int(0.35 * rs.dense_flops(p.seg_bounds, p.n_q_heads)), t_probe=rs.probe_flops(p.seg_bounds, p.n_q_heads),
        alpha=1.0, delta_q=calib["delta_q"], cert_max=0.5, beta=2.0, e=e))
    assert np.array_equal(got, want)


def test_calibration_command_line_on_synthetic_layers(tmp_path, capsys):
    """The offline calibration entry point end to end (seeded config-3 / config-4 recipe layers at a small length)."""
    import json
    out = tmp_path / "calibration.json"
    assert CALIB.main(["--n", "8192", "--layers", "1", "--held-out", "1", "--q", "0.9", "--out", str(out)]) == 0
    res = json.loads(out.read_text())
    assert res["n"] == 8192 and res["n_records"] == 32 * 12
    assert 0.0 <= res["delta_q"] < 1.0 and res["coverage_in_domain"]["mass"] >= 0.9
    assert res["coverage_in_domain"]["rows_exact_mass"] == 1.0          # Eq. 5 with the exact mass holds on every row
    for dom in ("same_recipe", "segmented"):
        assert res[f"coverage_held_out_{dom}"]["n"] > 0
    # the result installs into a layer
    layer = rs.RoutedPrefillLayer(rs.Problem(32, 8, 8192), None, rs.RouteConfig())
    layer.use_calibration(res, beta=1.0)
    assert layer.cfg.delta_q == res["delta_q"] and layer.cfg.beta == 1.0
