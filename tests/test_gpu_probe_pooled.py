"""GPU parity: rs_probe_pooled (Eq. 3 in its general form: mixture of query rows, pooled keys, descriptors) against
the oracle.

Tolerance: probabilities and masses within 2e-4 relative with an absolute floor of 1e-6 (fp32 pooled means and dot
products, fast exponentials), log-sum-exp within 1e-4, descriptors within 1e-4 absolute.
"""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import dev_bf16, f64_heads
from oracle import probe as OP
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu


def run(L, p, g, rows_per_seg, sub_bounds):
    Q, K = dev_bf16(L["Q"]), dev_bf16(L["K"])
    S, Hq, n = p.n_segments, p.n_q_heads, p.n_keys
    r = len(rows_per_seg[0])
    f32 = dict(dtype=torch.float32, device="cuda")
    rows = torch.tensor(rows_per_seg, dtype=torch.int32, device="cuda")
    n_sub = len(sub_bounds) - 1
    out = dict(A=torch.full((S, Hq, r, n // g), 3.0, **f32), lse=torch.zeros((S, Hq, r), **f32),
               col=torch.zeros((S, Hq, n_sub, n // g), **f32), diag=torch.zeros((S, Hq, n_sub, n // g), **f32),
               descr=torch.zeros((S, Hq, 4), **f32))
    scratch = torch.zeros(rs.rs_probe_pooled_scratch_floats(p, r), **f32)
    st = rs.new_status()
    rs.rs_probe_pooled(p, Q, K, rows, g, sub_bounds, out["A"], out["lse"], out["col"], out["diag"], out["descr"], scratch, st)
    rs.check_status(st, "pooled probe")
    return {k: v.cpu().numpy() for k, v in out.items()}


def close(a, b, rtol=2e-4, floor=1e-6):
    return np.all(np.abs(a - b) <= rtol * np.abs(b) + floor)


@pytest.mark.parametrize("n,Hq,Hkv,bounds,g", [(1024, 4, 1, None, 8), (1088, 4, 2, [0, 320, 1088], 16),
                                               (2048, 8, 2, None, 64), (704, 2, 2, [0, 64, 704], 4), (512, 3, 1, None, 1)])
def test_pooled_probe_matches_oracle(n, Hq, Hkv, bounds, g):
    L = make_layer(tiny_spec(77 + n + g, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
    rows = [rs.mixture_rows(p.seg_bounds[s], p.seg_bounds[s + 1]) for s in range(p.n_segments)]
    sub = [0, 32, 48, 64]
    got = run(L, p, g, rows, sub)
    Qs, Ks, _ = f64_heads(L)
    G = Hq // Hkv
    for s in range(p.n_segments):
        q1 = p.seg_bounds[s + 1]
        assert rows[s] == OP.mixture_rows(p.seg_bounds[s], q1).tolist()        # both sides use the same mixture
        for h in range(Hq):
            want = OP.pooled_probe(Qs[h], Ks[h // G], np.asarray(rows[s]), g, q1, sub)
            nbg = q1 // g
            assert close(got["A"][s, h][:, :nbg], want.A), (s, h)
            assert np.all(got["A"][s, h][:, nbg:] == 0)
            assert np.allclose(got["lse"][s, h], want.lse, atol=1e-4), (s, h)
            assert close(got["col"][s, h][:, :nbg], want.colmass), (s, h)
            assert close(got["diag"][s, h][:, :nbg], want.diagmass), (s, h)
            d = got["descr"][s, h]
            assert abs(d[0] - want.entropy) < 1e-4 and abs(d[1] - want.local_conc) < 1e-4, (s, h, d, want.entropy)
            assert abs(d[2] - want.agreement) < 1e-4, (s, h, d[2], want.agreement)
            assert abs(d[3] - np.mean([i // g + 1 for i in rows[s]])) < 1e-3


def test_pooled_probe_fewer_rows_and_one_subset():
    n, Hq, Hkv, g = 640, 2, 1, 32
    L = make_layer(tiny_spec(5, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n)
    rows = [list(range(n - 16, n)) + [5, 100, 333]]                  # 19 rows, one subset: agreement is 1 by definition
    got = run(L, p, g, rows, [0, 19])
    Qs, Ks, _ = f64_heads(L)
    for h in range(Hq):
        want = OP.pooled_probe(Qs[h], Ks[0], np.asarray(rows[0]), g, n, [0, 19])
        assert close(got["A"][0, h], want.A) and close(got["col"][0, h], want.colmass)
        assert abs(got["descr"][0, h][2] - 1.0) < 1e-6


def test_pooled_probe_rejects_bad_arguments():
    p = rs.Problem(8, 1, 256)                                          # 8 query heads per KV head: unsupported here
    f32 = dict(dtype=torch.float32, device="cuda")
    z = torch.zeros(16, **f32)
    rows = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    q = torch.zeros((8, 256, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rs.RouteSparseError):
        rs.rs_probe_pooled(p, q, q, rows, 8, [0, 4], z, z, z, z, z, z, rs.new_status())
    p = rs.Problem(2, 1, 256)
    with pytest.raises(rs.RouteSparseError):
        rs.rs_probe_pooled(p, q, q, rows, 24, [0, 4], z, z, z, z, z, z, rs.new_status())      # 24 does not divide 64
    with pytest.raises(rs.RouteSparseError):
        rs.rs_probe_pooled(p, q, q, rows, 8, [0, 3], z, z, z, z, z, z, rs.new_status())       # subsets do not cover r
