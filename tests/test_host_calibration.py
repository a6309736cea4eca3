"""The library's host functions for the offline calibration (Section 3.5) and the measured cost table (Section 3.1),
called through the C ABI on the CPU: against the oracle (itself pinned to scikit-learn), scipy's non-negative least
squares and hand-computed cases.  No GPU needed."""
import numpy as np
from scipy.optimize import nnls

import paper_2608_29058_b200 as rs
from oracle import calibration as OC


def _records(n=300, seed=0):
    rng = np.random.default_rng(seed)
    X = rng.uniform(0, 1, (n, 6))
    true_w = np.array([0.3, 0.1, 0.0, 0.0, 0.05, 0.02])
    y = np.clip(X @ true_w + rng.normal(0, 0.02, n), 0, None)
    res = rng.normal(-0.03, 0.05, n)
    return X, y, res


def test_fit_against_the_oracle_and_scipy():
    for seed in range(4):
        X, y, res = _records(seed=seed)
        dq, w, bz, be = rs.rs_calibration_fit(X, y, res, 0.9, max_breakpoints=10 ** 6)
        assert dq == OC.one_sided_quantile(res, 0.9)
        w_ref, _ = nnls(X, y)
        assert np.allclose(w, w_ref, atol=1e-7)
        assert min(w) >= 0
        # the step function of the target on z = X w is the oracle's isotonic fit (== scikit-learn's, pinned there)
        oz, oe = OC.isotonic_fit(X @ np.array(w), y)
        assert len(bz) == len(oz) and np.allclose(bz, oz, atol=0) and np.allclose(be, oe, rtol=1e-12, atol=1e-15)
        assert np.all(np.diff(be) >= 0) and np.all(np.diff(bz) > 0)


def test_quantile_by_counting_and_the_floor_at_zero():
    X, y, _ = _records(50)
    res = np.arange(50) / 100.0 - 0.2                       # -0.2 .. 0.29
    for q in (0.1, 0.5, 0.9, 1.0):
        dq = rs.rs_calibration_fit(X, y, res, q)[0]
        k = int(np.ceil(q * 50))
        assert dq == max(0.0, np.sort(res)[k - 1])
        assert (res <= dq + 1e-15).mean() >= q or dq == 0.0
    assert rs.rs_calibration_fit(X, y, -np.ones(50), 0.9)[0] == 0.0


def test_thinning_keeps_a_monotone_table_of_the_asked_size():
    X, y, res = _records(400, seed=9)
    _, w, bz, be = rs.rs_calibration_fit(X, y, res, 0.9, max_breakpoints=8)
    assert len(bz) <= 8 and np.all(np.diff(be) >= 0) and np.all(np.diff(bz) > 0)
    _, w2, bz2, be2 = rs.rs_calibration_fit(X, y, res, 0.9, max_breakpoints=10 ** 6)
    assert set(bz) <= set(bz2) and bz[0] == bz2[0]          # thinning only drops breakpoints, never the first


def test_hand_computed_isotonic_case():
    # one feature, weight forced by the data: y = (1, 3, 2, 4) at z = (1, 2, 3, 4) -> pooled (1, 2.5, 2.5, 4)
    X = np.array([[1.0], [2.0], [3.0], [4.0]])
    y = np.array([1.0, 3.0, 2.0, 4.0])
    _, w, bz, be = rs.rs_calibration_fit(X, y, np.zeros(4), 0.5)
    assert np.allclose(np.array(bz) / w[0], [1.0, 2.0, 4.0]) and np.allclose(be, [1.0, 2.5, 4.0])


def test_cost_table_splits_the_measured_time_by_pair_counts():
    pairs = np.array([[100, 10], [300, 30], [0, 0]], dtype=np.uint64)
    table = rs.rs_cost_table_from_times([4.0, 1.0], pairs)
    assert table[:, 0].tolist() == [1000000, 3000000, 1] and table[:, 1].tolist() == [250000, 750000, 1]
    assert abs(int(table[:2, 0].sum()) - 4_000_000) <= 1
