"""GPU parity: rs_probe against the oracle's probe (Eq. 3, last-64-query form).

Tolerance: probe scores within 1e-3 relative (fp32 accumulation, ex2.approx) with an absolute floor of 1e-7
for entries that underflow; pooled means and V_max within 1e-5 relative.
"""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import dev_bf16, f64_heads
from oracle import probe as OP
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu


def run_probe(L, p):
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    S, Hq, Hkv, n = p.n_segments, p.n_q_heads, p.n_kv_heads, p.n_keys
    f32 = dict(dtype=torch.float32, device="cuda")
    out = dict(vert=torch.full((S, Hq, 4, n), 7.0, **f32), slash=torch.full((S, Hq, 4, n), 7.0, **f32),
               lse=torch.zeros((Hq, S, 64), **f32), qpool=torch.zeros((Hq, n // 64, 128), **f32),
               kpool=torch.zeros((Hkv, n // 64, 128), **f32), vmax=torch.zeros((S, Hkv), **f32))
    ws = rs.new_workspace(p, None)
    st = rs.new_status()
    rs.rs_probe(p, Q, K, V, out["vert"], out["slash"], out["lse"], out["qpool"], out["kpool"], out["vmax"], None, ws, st)
    rs.check_status(st, "probe")
    return {k: v.cpu().numpy() for k, v in out.items()}


def close(a, b, rtol=1e-3, floor=1e-7):
    return np.all(np.abs(a - b) <= rtol * np.abs(b) + floor)


@pytest.mark.parametrize("n,Hq,Hkv,bounds", [(256, 2, 1, None), (1088, 4, 2, [0, 320, 1088]), (704, 4, 1, None),
                                             (448, 2, 2, [0, 64, 448]), (640, 8, 1, None)])
def test_probe_matches_oracle(n, Hq, Hkv, bounds):
    L = make_layer(tiny_spec(31 + n, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
    got = run_probe(L, p)
    Qs, Ks, Vs = f64_heads(L)
    G = Hq // Hkv
    for s in range(p.n_segments):
        q1 = p.seg_bounds[s + 1]
        for h in range(Hq):
            pr = OP.probe_rows(Qs[h], Ks[h // G], q1)
            assert close(got["lse"][h, s], pr.lse, 1e-5, 1e-4), (s, h)
            assert close(got["vert"][s, h][:, :q1], pr.vert), (s, h)
            assert close(got["slash"][s, h][:, :q1], pr.slash), (s, h)
            assert np.all(got["vert"][s, h][:, q1:] == 0) and np.all(got["slash"][s, h][:, q1:] == 0)
            assert abs(got["vert"][s, h].sum() - 64) < 1e-2 and abs(got["slash"][s, h].sum() - 64) < 1e-2
        for g in range(Hkv):
            _, vmax = OP.value_norms(Vs[g], q1)
            assert abs(got["vmax"][s, g] - vmax) <= 1e-5 * vmax
    for h in range(Hq):
        assert np.allclose(got["qpool"][h], OP.pool_mean(Qs[h]), rtol=1e-5, atol=1e-6)
    for g in range(Hkv):
        assert np.allclose(got["kpool"][g], OP.pool_mean(Ks[g]), rtol=1e-5, atol=1e-6)


def test_probe_is_deterministic():
    L = make_layer(tiny_spec(77, 1024, 4, 1))
    p = rs.Problem(4, 1, 1024)
    a, b = run_probe(L, p), run_probe(L, p)
    for k in a:
        assert np.array_equal(a[k], b[k]), k


def test_probe_descriptors_match_oracle():
    """descr output of rs_probe: entropy and local-band mass of the exact probe rows (Section 3.2)."""
    for n, Hq, Hkv, bounds in ((2304, 4, 2, None), (1088, 4, 2, [0, 320, 1088]), (2048 + 1280, 2, 1, None)):
        L = make_layer(tiny_spec(55 + n, n, Hq, Hkv))
        p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
        Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
        S = p.n_segments
        f32 = dict(dtype=torch.float32, device="cuda")
        vert = torch.zeros((S, Hq, 4, n), **f32); slash = torch.zeros((S, Hq, 4, n), **f32)
        lse = torch.zeros((Hq, S, 64), **f32); descr = torch.full((S, Hq, 2), -1.0, **f32)
        st = rs.new_status()
        rs.rs_probe(p, Q, K, V, vert, slash, lse, None, None, None, descr, rs.new_workspace(p, None), st)
        rs.check_status(st, "probe with descriptors")
        got = descr.cpu().numpy()
        Qs, Ks, _ = f64_heads(L)
        for s in range(S):
            for h in range(Hq):
                pr = OP.probe_rows(Qs[h], Ks[h // (Hq // Hkv)], p.seg_bounds[s + 1])
                assert abs(got[s, h, 0] - pr.entropy) < 2e-3 * max(1.0, pr.entropy), (n, s, h, got[s, h, 0], pr.entropy)
                assert abs(got[s, h, 1] - pr.local_conc) < 1e-3, (n, s, h, got[s, h, 1], pr.local_conc)


def test_lazy_query_pooling_equals_full_pooling_where_it_is_read():
    """RS_PROBE_QPOOL_LAST_ONLY fills the last query block of every segment; rs_pool_queries adds every block of the
    heads routed to block-sparse; together they hold the same bits as the full pooling wherever anything reads them."""
    n, Hq, Hkv = 1088, 4, 2
    L = make_layer(tiny_spec(17, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, [0, 320, 1088])
    full = run_probe(L, p)["qpool"]
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    f32 = dict(dtype=torch.float32, device="cuda")
    S = p.n_segments
    vert = torch.zeros((S, Hq, 4, n), **f32); slash = torch.zeros((S, Hq, 4, n), **f32); lse = torch.zeros((Hq, S, 64), **f32)
    qpool = torch.full((Hq, n // 64, 128), 123.0, **f32)
    st = rs.new_status()
    rs.rs_probe(p, Q, K, V, vert, slash, lse, qpool, None, None, None, rs.new_workspace(p, None), st,
                flags=rs.RS_PROBE_QPOOL_LAST_ONLY)
    got = qpool.cpu().numpy()
    for s in range(S):
        qb = p.seg_bounds[s + 1] // 64 - 1
        assert np.array_equal(got[:, qb], full[:, qb])
    assert np.all(got[:, 0] == 123.0)                                   # untouched elsewhere
    lib = rs.make_library([(rs.RS_A_SHAPE, 64, 128), (rs.RS_BLOCK_SPARSE, 3, 0), (rs.RS_DENSE, 0, 0)])
    # items = (segment, head): heads 1 and 2 go block-sparse in segment 0, head 3 in segment 1
    choice = torch.tensor([0, 1, 1, 2, 0, 2, 0, 1], dtype=torch.int32, device="cuda")
    rs.rs_pool_queries(p, Q, lib, choice, qpool, st)
    rs.check_status(st, "lazy pooling")
    got = qpool.cpu().numpy()
    seg0 = slice(0, 320 // 64); seg1 = slice(320 // 64, n // 64)
    for h in (1, 2):
        assert np.array_equal(got[h, seg0], full[h, seg0])
    assert np.array_equal(got[3, seg1], full[3, seg1])
    assert np.all(got[0, 1:4] == 123.0) and np.all(got[3, 0:4] == 123.0)   # heads not routed to block-sparse stay untouched
    rs.rs_pool_queries(p, Q, None, None, qpool, st)                     # no choice: every head
    assert np.array_equal(qpool.cpu().numpy(), full)


@pytest.mark.parametrize("n,Hq,Hkv,bounds", [(1088, 8, 1, [0, 320, 1088]), (640, 6, 2, None), (4096, 8, 2, [0, 64, 4096])])
def test_last_query_block_from_the_staged_probe_rows(n, Hq, Hkv, bounds):
    """With RS_PROBE_QPOOL_LAST_ONLY the second pass pools each segment's last query block from the probe rows it has
    staged (head groups larger than one CTA's four head slots included); V_max comes from the same pass.  Both must
    hold the bits of the full pooling and of the call without the flag."""
    L = make_layer(tiny_spec(77 + n, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
    full = run_probe(L, p)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    f32 = dict(dtype=torch.float32, device="cuda")
    S = p.n_segments
    vert = torch.zeros((S, Hq, 4, n), **f32); slash = torch.zeros((S, Hq, 4, n), **f32); lse = torch.zeros((Hq, S, 64), **f32)
    qpool = torch.full((Hq, n // 64, 128), -5.0, **f32)
    vmax = torch.zeros((S, Hkv), **f32)
    st = rs.new_status()
    rs.rs_probe(p, Q, K, V, vert, slash, lse, qpool, None, vmax, None, rs.new_workspace(p, None), st,
                flags=rs.RS_PROBE_QPOOL_LAST_ONLY)
    rs.check_status(st, "probe, last block only")
    got = qpool.cpu().numpy()
    last = [p.seg_bounds[s + 1] // 64 - 1 for s in range(S)]
    for qb in last:
        assert np.array_equal(got[:, qb], full["qpool"][:, qb])
    others = [qb for qb in range(n // 64) if qb not in last]
    assert np.all(got[:, others] == -5.0)
    assert np.array_equal(vmax.cpu().numpy(), full["vmax"])
    assert np.array_equal(vert.cpu().numpy(), full["vert"]) and np.array_equal(slash.cpu().numpy(), full["slash"])
