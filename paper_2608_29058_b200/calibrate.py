"""Offline calibration (Section 3.5): dense audits of calibration layers give the true retained mass and the output
error of every (head, candidate); from them come the one-sided residual quantile delta_q of the probe's mass estimate,
the coverage of the resulting empirical certificate (Eq. 5 with m_low = max(0, m_hat - delta_q)), and the monotone
predictor e of Eq. 4.  Every attention launch, certificate and row error runs in the library's kernels and the statistics over
the few hundred (head, candidate) records in its host function rs_calibration_fit; this module only gathers records.

Not part of the hot path: run once per model / library / length bucket, then RoutedPrefillLayer.use_calibration().

    python -m paper_2608_29058_b200.calibrate --n 16384 --layers 3 --held-out 2 --out calibration.json
"""
from __future__ import annotations

import argparse
import json
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as rs
from .pipeline import RoutedPrefillLayer, RouteConfig

FEATURES = ("1 - m_hat", "u", "entropy", "1 - local", "1 - agreement", "1 - pairs / dense pairs")


# ------------------------------------------------------------------------------------------ audits
def audit_layer(Q, K, V, problem: rs.Problem, library=None, g: int = 64) -> List[Dict]:
    """One record per (item, sparse candidate): m_hat, u, m_true, mean row error, V_max, features, coverage of rows."""
    dev = Q.device
    p = problem
    layer = RoutedPrefillLayer(p, library, RouteConfig(), device=dev)
    layer.probe(Q, K, V)
    layer.evaluate_candidates()
    descr = layer.pooled_probe(Q, K, g=g).reshape(p.n_items, 4).cpu().numpy()
    Hq, n = p.n_q_heads, p.n_keys
    O_d = torch.empty_like(layer.O)
    lse_d = torch.empty((Hq, n), dtype=torch.float32, device=dev)
    rs.rs_dense_prefill_attn(p, Q, K, V, O_d, lse_d, None, None, layer.ws, layer.status)
    stats = layer.stats.cpu().numpy()
    vmax = layer.vmax.cpu().numpy()                    # [n_seg][Hkv]
    err = torch.empty(Hq * n, dtype=torch.float32, device=dev)
    group = Hq // p.n_kv_heads
    records = []
    for c, cand in enumerate(layer.cands):
        if cand[0] == rs.RS_DENSE:
            continue
        layer.choice.fill_(c)
        layer.materialise(reuse_evaluation=True)
        layer.attention(Q, K, V)
        rs.rs_output_error(O_d, layer.O, err, None, layer.status)
        err_rows = err.view(Hq, n)
        for s in range(p.n_segments):
            q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
            rows = torch.arange(q0, q1, dtype=torch.int32, device=dev)
            m_row = torch.empty((Hq, q1 - q0), dtype=torch.float32, device=dev)
            cert_row = torch.empty_like(m_row)
            m_head = torch.empty(Hq, dtype=torch.float32, device=dev)
            vmax_s = layer.vmax[s].contiguous()
            rs.rs_certificate(Hq, p.n_kv_heads, n, layer.lse_sel, lse_d[:, q0:q1].contiguous(), rows, vmax_s, None, 0.0,
                              m_row, cert_row, None, m_head, None, layer.status)
            e_seg = err_rows[:, q0:q1]
            mean_err = e_seg.mean(dim=1).cpu().numpy()
            # Eq. 5 row by row with the exact mass; bf16 rounding of the two outputs is allowed for (2^-7 of the norm scale)
            slack = 2.0 ** -7 * vmax_s.repeat_interleave(group)[:, None]
            row_cov = (e_seg <= cert_row + slack).float().mean(dim=1).cpu().numpy()
            m_true = m_head.cpu().numpy()
            dense_pairs = (q1 * (q1 + 1) - q0 * (q0 + 1)) // 2
            for h in range(Hq):
                item = s * Hq + h
                cov = stats[item, c, :4].astype(np.uint64)
                mg = cov.astype(np.float64) / (16.0 * 2.0 ** 32)
                m_hat = float(cov.sum(dtype=np.uint64)) / (64.0 * 2.0 ** 32)
                u = float(mg.max() - mg.min())
                d = descr[item]
                feats = [1.0 - m_hat, u, float(d[0]), 1.0 - float(d[1]), 1.0 - float(d[2]),
                         1.0 - float(stats[item, c, 4]) / float(dense_pairs)]
                records.append(dict(item=item, cand=c, m_hat=m_hat, u=u, m_true=float(m_true[h]),
                                    mean_err=float(mean_err[h]), vmax=float(vmax[s, h // group]),
                                    row_coverage=float(row_cov[h]), features=feats))
    rs.check_status(layer.status, "calibration audit")
    return records


def coverage(records: List[Dict], delta_q: float) -> Dict[str, float]:
    """Share of records whose true mass is at least m_hat - delta_q, and whose empirical certificate
    2 (1 - max(0, m_hat - delta_q)) V_max is at least the mean row error."""
    if not records:
        return {"mass": float("nan"), "certificate": float("nan"), "rows_exact_mass": float("nan"), "n": 0}
    mass = np.mean([r["m_true"] >= r["m_hat"] - delta_q for r in records])
    cert = np.mean([r["mean_err"] <= 2.0 * (1.0 - max(0.0, r["m_hat"] - delta_q)) * r["vmax"] for r in records])
    rows = np.mean([r["row_coverage"] for r in records])
    return {"mass": float(mass), "certificate": float(cert), "rows_exact_mass": float(rows), "n": len(records)}


def calibrate(calibration_records: List[Dict], held_out: Optional[Dict[str, List[Dict]]] = None, q: float = 0.9,
              g: int = 64) -> Dict:
    """delta_q, certificate coverage (in-domain and per held-out domain) and the predictor e from audit records."""
    res = [r["m_hat"] - r["m_true"] for r in calibration_records]
    X = np.array([r["features"] for r in calibration_records], dtype=np.float64)
    y = np.array([r["mean_err"] / max(r["vmax"], 1e-30) for r in calibration_records], dtype=np.float64)
    delta_q, w, bp_z, bp_e = rs.rs_calibration_fit(X, y, res, q)          # the statistics run in the library
    w = np.array(w)
    fit = np.array([max([e for zk, e in zip(bp_z, bp_e) if zk <= z], default=0.0) for z in X @ w])
    out = {"q": q, "delta_q": delta_q, "n_records": len(calibration_records),
           "residual_mean": float(np.mean(res)), "residual_max": float(np.max(res)),
           "coverage_in_domain": coverage(calibration_records, delta_q),
           "coverage_without_delta": coverage(calibration_records, 0.0),
           "regressor": {"g": g, "features": list(FEATURES), "w": [float(x) for x in w], "bp_z": bp_z, "bp_e": bp_e,
                         "target": "mean row error / V_max", "fit_rmse": float(np.sqrt(np.mean((fit - y) ** 2))),
                         "target_std": float(np.std(y))}}
    for name, recs in (held_out or {}).items():
        out[f"coverage_held_out_{name}"] = coverage(recs, delta_q)
    return out


# ------------------------------------------------------------------------------------------ command line (synthetic layers)
def _synthetic_layer(spec, dev):
    from synth import make_layer
    L = make_layer(spec)
    to_dev = lambda bits: torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
    p = rs.Problem(spec.n_q_heads, spec.n_kv_heads, spec.n, [int(x) for x in L["seg_bounds"]])
    return to_dev(L["Q"]), to_dev(L["K"]), to_dev(L["V"]), p


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--n", type=int, default=16384)
    ap.add_argument("--layers", type=int, default=3, help="calibration layers (seeded, config-3 recipe)")
    ap.add_argument("--held-out", type=int, default=2, help="held-out layers per held-out domain")
    ap.add_argument("--q", type=float, default=0.9)
    ap.add_argument("--g", type=int, default=64)
    ap.add_argument("--out", type=str, default=None)
    args = ap.parse_args(argv)
    from synth import config3_spec, config4_layer_spec
    dev = torch.device("cuda", 0)
    recs: List[Dict] = []
    for k in range(args.layers):                       # in-domain: the config-3 recipe under different seeds
        recs += audit_layer(*_synthetic_layer(config3_spec(args.n, seed_offset=5000 + k), dev), g=args.g)
    held: Dict[str, List[Dict]] = {"same_recipe": [], "segmented": []}
    for k in range(args.held_out):
        held["same_recipe"] += audit_layer(*_synthetic_layer(config3_spec(args.n, seed_offset=9000 + k), dev), g=args.g)
        held["segmented"] += audit_layer(*_synthetic_layer(config4_layer_spec(k, args.n, seg_len=args.n // 4), dev), g=args.g)
    out = calibrate(recs, held, q=args.q, g=args.g)
    out["n"] = args.n
    text = json.dumps(out)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text + "\n")
    print(text)
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
