"""GPU parity: rs_certificate against the oracle (Eq. 5), and the bound against the true error."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from oracle import certificate as CT

pytestmark = pytest.mark.gpu


def test_certificate_matches_oracle():
    rng = np.random.default_rng(0)
    Hq, n, R = 3, 512, 200
    lse_full = rng.uniform(2, 8, (Hq, R)).astype(np.float32)
    rows = np.sort(rng.choice(n, R, replace=False)).astype(np.int32)
    lse_sel = np.zeros((Hq, n), np.float32)
    lse_sel[:, rows] = lse_full - rng.exponential(0.05, (Hq, R)).astype(np.float32)
    lse_sel[0, rows[:5]] = lse_full[0, :5] + 1e-6          # rounding may put lse_sel a hair above: m clamps to 1
    onorm = rng.uniform(0, 10, (Hq, n)).astype(np.float32)
    vmax = np.float32([13.5, 12.0, 14.25])
    t = lambda a: torch.from_numpy(a).cuda()
    out = [torch.zeros((Hq, R), device="cuda") for _ in range(3)] + [torch.zeros(Hq, device="cuda"), torch.zeros((Hq, 2), device="cuda")]
    rs.rs_certificate(Hq, Hq, n, t(lse_sel), t(lse_full), t(rows), t(vmax), t(onorm), 0.01, *out, None)
    m_row, cert_row, tight, m_head, cert_head = [o.cpu().numpy() for o in out]
    for h in range(Hq):
        m, cert, tg, mh, ch, cm = CT.certificate(lse_sel[h, rows], lse_full[h], vmax[h], onorm[h, rows], 0.01)
        assert np.allclose(m_row[h], m, rtol=1e-5, atol=1e-6)
        assert np.allclose(cert_row[h], cert, rtol=1e-4, atol=1e-5)
        assert np.allclose(tight[h], tg, rtol=1e-4, atol=1e-5)
        assert abs(m_head[h] - mh) < 1e-6 and abs(cert_head[h, 0] - ch) < 1e-4 and abs(cert_head[h, 1] - cm) < 1e-4
    assert np.all(m_row <= 1.0) and np.all(cert_row >= 0)


def test_row_ids_outside_the_sequence_are_reported_not_read():
    """A row id outside [0, n_keys) is never dereferenced: NaN outputs for that row, the head-level mean over the valid
    rows only, and RS_ERR_INVALID_ARG in the status words."""
    rng = np.random.default_rng(1)
    Hq, n, R = 2, 256, 40
    rows = np.sort(rng.choice(n, R, replace=False)).astype(np.int32)
    lse_full = rng.uniform(2, 8, (Hq, R)).astype(np.float32)
    lse_sel = np.zeros((Hq, n), np.float32)
    lse_sel[:, rows] = lse_full - rng.exponential(0.05, (Hq, R)).astype(np.float32)
    bad = rows.copy()
    bad[3], bad[17] = n, -1
    vmax = np.float32([3.0, 4.0])
    t = lambda a: torch.from_numpy(a).cuda()
    m_row, m_head = torch.zeros((Hq, R), device="cuda"), torch.zeros(Hq, device="cuda")
    st = rs.new_status()
    rs.rs_certificate(Hq, Hq, n, t(lse_sel), t(lse_full), t(bad), t(vmax), None, 0.0, m_row, None, None, m_head, None, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == -1
    got = m_row.cpu().numpy()
    assert np.isnan(got[:, [3, 17]]).all()
    ok = np.ones(R, bool); ok[[3, 17]] = False
    for h in range(Hq):
        m = CT.certificate(lse_sel[h, rows[ok]], lse_full[h, ok], vmax[h], None, 0.0)[0]
        assert np.allclose(got[h, ok], m, rtol=1e-5, atol=1e-6)
        assert abs(float(m_head[h]) - float(np.mean(m))) < 1e-6


def test_bounded_wait_gives_up_and_reports():
    """A device-side wait that nothing satisfies runs out by itself; the status words say so and the context lives on."""
    st = rs.new_status()
    rs.rs_selftest_wait_timeout(st, 2000)
    torch.cuda.synchronize()
    words = st.cpu().tolist()
    assert words[0] == -6 and words[1] == 99
    with pytest.raises(rs.RouteSparseError, match="bounded device-side wait"):
        rs.check_status(st, "self test")
    assert float((torch.ones(4, device="cuda") * 2).sum()) == 8.0       # the device still answers
