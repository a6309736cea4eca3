"""Pins for the oracle's calibration pieces (Section 3.5; predictor e of Eq. 4). CPU only."""
import numpy as np

from oracle import calibration as CAL
from oracle import patterns as PT
from oracle import routing as RT


def test_isotonic_fit_equals_scikit_learn():
    from sklearn.isotonic import IsotonicRegression
    rng = np.random.default_rng(0)
    for n in (1, 2, 7, 50, 300):
        z = np.round(rng.random(n), 2)                 # rounded: ties occur
        y = z * 0.7 + 0.2 * rng.standard_normal(n)
        bz, be = CAL.isotonic_fit(z, y)
        assert np.all(np.diff(bz) > 0) and np.all(np.diff(be) >= 0)
        ref = IsotonicRegression(increasing=True, out_of_bounds="clip").fit(z, y)
        for zz in np.unique(z):
            assert abs(CAL.step_eval(bz, be, float(zz)) - float(ref.predict([zz])[0])) < 1e-12, (n, zz)
    # already monotone data is reproduced, a decreasing pair is pooled to its mean
    bz, be = CAL.isotonic_fit([0.1, 0.2, 0.3], [1.0, 2.0, 3.0])
    assert np.allclose(be, [1, 2, 3])
    bz, be = CAL.isotonic_fit([0.1, 0.2], [3.0, 1.0])
    assert len(be) == 1 and be[0] == 2.0 and bz[0] == 0.1
    assert CAL.step_eval(bz, be, 0.05) == 0.0 and CAL.step_eval(bz, be, 5.0) == 2.0


def test_one_sided_quantile_by_counting():
    r = [0.3, -0.2, 0.05, 0.1, 0.0, -0.4, 0.2, 0.15, 0.01, 0.02]
    for q in (0.5, 0.9, 0.95, 1.0):
        d = CAL.one_sided_quantile(r, q)
        assert d >= 0.0 and np.mean(np.asarray(r) <= d) >= q
        smaller = [x for x in sorted(r) if 0 <= x < d]   # no smaller non-negative candidate satisfies the count
        assert all(np.mean(np.asarray(r) <= x) < q for x in smaller)
    assert CAL.one_sided_quantile([-0.3, -0.1], 0.9) == 0.0 and CAL.one_sided_quantile([], 0.9) == 0.0


def test_true_mass_and_coverage_rule():
    lse_full = np.log(np.array([4.0, 10.0, 2.0]))
    lse_sel = np.log(np.array([2.0, 10.0, 1.0]))
    assert abs(CAL.true_mass(lse_sel, lse_full) - (0.5 + 1.0 + 0.5) / 3) < 1e-12
    assert CAL.certificate_covers(0.75, 0.0, 2.0, 1.0) and not CAL.certificate_covers(0.75, 0.0, 2.0, 1.01)
    assert CAL.certificate_covers(0.75, 0.25, 2.0, 2.0) and not CAL.certificate_covers(0.75, 0.25, 2.0, 2.01)


def test_predictor_is_monotone_and_enters_the_risk():
    lib = [PT.Candidate(PT.A_SHAPE, 64, 128), PT.Candidate(PT.A_SHAPE, 64, 256), PT.Candidate(PT.DENSE)]
    one = np.uint64(PT.FX_ONE)
    cov = np.zeros((2, 3, 4), dtype=np.uint64)
    cov[0, 0] = [one * 12, one * 12, one * 10, one * 14]       # m_hat 0.75, u 0.25
    cov[0, 1] = [one * 15] * 4                                  # m_hat 0.9375, u 0
    cov[1, 0] = [one * 8] * 4
    cov[1, 1] = [one * 16] * 4
    pairs = np.array([[1000, 2000, 8256], [1000, 2000, 8256]])
    descr = np.array([[0.5, 0.9, 0.8, 3.0], [0.9, 0.2, 0.3, 3.0]], dtype=np.float32)
    w = [1.0, 0.5, 0.2, 0.1, 0.3, 0.05]
    bz, be = np.array([0.0, 0.4, 0.8]), np.array([0.0, 0.1, 0.5])
    e = CAL.regressor_eval(lib, cov, pairs, descr, [(0, 128), (0, 128)], w, bz, be)
    assert np.all(e[:, 2] == 0.0)                                        # dense
    assert e[0, 1] <= e[0, 0] and e[1, 1] <= e[1, 0]                     # more coverage, more pairs: not riskier
    f = CAL.features(cov[0, 0], 1000, descr[0], 0, 128)
    assert abs(f[0] - 0.25) < 1e-12 and abs(f[1] - 0.25) < 1e-12 and abs(f[5] - (1 - 1000 / 8256)) < 1e-12
    # worse descriptors never lower e
    worse = descr.copy(); worse[:, 0] = 1.0; worse[:, 1] = 0.0; worse[:, 2] = 0.0
    e2 = CAL.regressor_eval(lib, cov, pairs, worse, [(0, 128), (0, 128)], w, bz, be)
    assert np.all(e2 >= e)
    # Eq. 4: R = (1 - m_hat) + alpha u + beta e
    R0, _ = RT.risks(lib, cov, 1.0)
    R1, _ = RT.risks(lib, cov, 1.0, 2.0, e)
    assert np.allclose(R1 - R0, 2.0 * e) and R1[0, 2] == 0.0
    # a large e on one substitution moves it to the other item: the budget forces exactly one item onto candidate 0
    cost = np.array([[100, 200, 800], [100, 200, 800]], dtype=np.int64)
    vmax = np.ones(2, dtype=np.float32)
    ch0, _ = RT.route(lib, cov, cost, vmax, RT.RouteParams(budget=300))
    ebig = np.zeros_like(e); ebig[0, 0] = 100.0
    ch1, _ = RT.route(lib, cov, cost, vmax, RT.RouteParams(budget=300, beta=1.0, e=ebig))
    assert list(ch0) == [0, 1] and list(ch1) == [1, 0]
