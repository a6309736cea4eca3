"""Pins for the oracle's certificate (Eq. 5). CPU only."""
import os

import numpy as np

from oracle import attention as A
from oracle import certificate as CT
from oracle import patterns as PT
from oracle import probe as P
from synth import bf16_bits_to_f64, make_layer, tiny_spec

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "eq5_two_key_case.txt")


def test_equality_case_from_golden_file():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        m, Vn, err = (float(x) for x in line.split())
        # two keys with logits chosen so that the exact row is a = (1 - m, m); key 1 is retained
        with np.errstate(divide="ignore"):
            lse_full = np.float32([np.logaddexp(np.log(1 - m), np.log(m))])
        lse_sel = np.float32([np.log(m)])
        mrow, cert, tight, m_head, cert_head, cert_max = CT.certificate(lse_sel, lse_full, Vn, np.float32([Vn]))
        assert abs(mrow[0] - m) < 1e-6 and abs(cert[0] - err) < 1e-5 and abs(tight[0] - err) < 1e-5
        v = np.array([[-Vn, 0.0], [Vn, 0.0]])
        a = np.array([1 - m, m])
        true_err = np.linalg.norm(a @ v - v[1])
        assert abs(true_err - err) < 1e-9
        assert abs(cert_head - err) < 1e-5 and abs(cert_max - err) < 1e-5


def test_l1_identity():
    rng = np.random.default_rng(0)
    a = rng.random(200)
    a /= a.sum()
    S = rng.random(200) < 0.4
    m = a[S].sum()
    at = np.where(S, a, 0) / m
    assert abs(np.abs(a - at).sum() - 2 * (1 - m)) < 1e-12


def test_certificate_bounds_true_error_on_every_row_and_pattern():
    L = make_layer(tiny_spec(21, 512, 2, 1))
    K, V = bf16_bits_to_f64(L["K"][0]), bf16_bits_to_f64(L["V"][0])
    for h in range(2):
        Q = bf16_bits_to_f64(L["Q"][h])
        O, lse = A.dense_attention(Q, K, V)
        pr = P.probe_rows(Q, K, 512)
        bs = P.block_scores(Q, K, 0, 512)
        _, vmax = P.value_norms(V, 512)
        for cand in (PT.Candidate(PT.A_SHAPE, 4, 32), PT.Candidate(PT.VERTICAL_SLASH, 16, 8),
                     PT.Candidate(PT.VERTICAL_SLASH, 16, 8, strict=True), PT.Candidate(PT.BLOCK_SPARSE, 2),
                     PT.Candidate(PT.DENSE)):
            ix = PT.build_indices(cand, 0, 512, pr.vert, pr.slash, bs)
            Om, lsel, onorm = A.masked_attention(Q, K, V, lambda r, nk: PT.mask_rows(ix, r, nk))
            m, cert, tight, m_head, cert_head, cert_max = CT.certificate(lsel, lse, vmax, onorm)
            err = np.linalg.norm(O.astype(np.float64) - Om.astype(np.float64), axis=1)
            assert np.all(cert + 1e-5 >= err), cand
            assert np.all(tight + 1e-5 >= err) and np.all(tight <= cert + 1e-9)
            if cand.pattern == PT.DENSE:
                assert np.all(cert == 0) and m_head == 1.0
            else:
                assert err.max() > 1e-3          # the sparse masks really do change the output
            # consistency of kernel-side mass and builder-side coverage on the probe rows
            if not cand.strict and cand.pattern != PT.DENSE:
                m_hat, _ = PT.m_hat_from_fx(PT.coverage_fx(ix, pr.vert, pr.slash))
                assert abs(m[-64:].mean() - m_hat) < 1e-5


def test_delta_q_lowers_the_mass():
    _, _, _, m_head, cert_head, _ = CT.certificate(np.float32([-0.1, -0.2]), np.float32([0, 0]), 2.0, None, 0.05)
    assert abs(cert_head - 2 * (1 - (m_head - 0.05)) * 2.0) < 1e-12
