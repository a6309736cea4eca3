"""GPU parity: the probe on the query mixture of Eq. 3 at key resolution (rs_probe_runs) and the vertical / slash lists
ranked by it (rs_build_indices_ranked) against the oracle."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import c_library, dev_bf16, f64_heads
from oracle import patterns as PT
from oracle import probe as OP
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu
C = PT.Candidate


def close(a, b, rtol=1e-3, floor=1e-7):
    return np.all(np.abs(a - b) <= rtol * np.abs(b) + floor)


def run_probe_runs(L, p, runs):
    Q, K = dev_bf16(L["Q"]), dev_bf16(L["K"])
    S, Hq, n = p.n_segments, p.n_q_heads, p.n_keys
    f32 = dict(dtype=torch.float32, device="cuda")
    vert, slash = torch.full((S, Hq, 4, n), 7.0, **f32), torch.full((S, Hq, 4, n), 7.0, **f32)
    lse = torch.zeros((Hq, S, 64), **f32)
    st = rs.new_status()
    rs.rs_probe_runs(p, Q, K, runs, vert, slash, lse, rs.new_workspace(p, None), st)
    rs.check_status(st, "probe on runs")
    return vert.cpu().numpy(), slash.cpu().numpy(), lse.cpu().numpy()


@pytest.mark.parametrize("n,Hq,Hkv,bounds", [(256, 2, 1, None), (1088, 4, 2, [0, 320, 1088]), (2304, 4, 1, None),
                                             (448, 2, 2, [0, 64, 448])])
def test_probe_on_mixture_runs_matches_oracle(n, Hq, Hkv, bounds):
    L = make_layer(tiny_spec(61 + n, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
    runs = [rs.rs_mixture_runs(p.seg_bounds[s], p.seg_bounds[s + 1]) for s in range(p.n_segments)]
    vert, slash, lse = run_probe_runs(L, p, runs)
    Qs, Ks, _ = f64_heads(L)
    G = Hq // Hkv
    for s in range(p.n_segments):
        q1 = p.seg_bounds[s + 1]
        assert runs[s] == OP.mixture_runs(p.seg_bounds[s], q1).tolist()
        for h in range(Hq):
            pr = OP.probe_rows(Qs[h], Ks[h // G], q1, runs[s])
            assert close(lse[h, s], pr.lse, 1e-5, 1e-4), (s, h)
            assert close(vert[s, h][:, :q1], pr.vert), (s, h)
            assert close(slash[s, h][:, :q1], pr.slash), (s, h)
            assert np.all(vert[s, h][:, q1:] == 0) and np.all(slash[s, h][:, q1:] == 0)
            assert abs(vert[s, h].sum() - 64) < 1e-2 and abs(slash[s, h].sum() - 64) < 1e-2


def test_runs_of_the_last_64_rows_give_the_ordinary_probe_bit_for_bit():
    n, Hq, Hkv = 1088, 4, 2
    L = make_layer(tiny_spec(5, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, [0, 320, 1088])
    runs = [[q1 - 64 + 16 * g for g in range(4)] for q1 in p.seg_bounds[1:]]
    vert, slash, lse = run_probe_runs(L, p, runs)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    f32 = dict(dtype=torch.float32, device="cuda")
    v2, s2, l2 = torch.zeros((2, Hq, 4, n), **f32), torch.zeros((2, Hq, 4, n), **f32), torch.zeros((Hq, 2, 64), **f32)
    st = rs.new_status()
    rs.rs_probe(p, Q, K, V, v2, s2, l2, None, None, None, None, rs.new_workspace(p, None), st)
    assert np.array_equal(vert, v2.cpu().numpy()) and np.array_equal(slash, s2.cpu().numpy()) and np.array_equal(lse, l2.cpu().numpy())


def test_lists_ranked_by_the_mixture_and_statistics_on_the_last_rows_are_bit_exact():
    """rs_build_indices_ranked: V and S are the oracle's top-k of the mixture's masses; coverage and pairs are the
    oracle's statistics of those lists measured on the last-64-row masses."""
    n, Hq, Hkv = 1344, 2, 1
    L = make_layer(tiny_spec(71, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, [0, 448, 1344])
    Qs, Ks, _ = f64_heads(L)
    lib = [C(PT.A_SHAPE, 8, 64), C(PT.VERTICAL_SLASH, 16, 24), C(PT.VERTICAL_SLASH, 40, 70), C(PT.DENSE)]
    lib_c = c_library(lib)
    S = p.n_segments
    vert = np.zeros((S, Hq, 4, n), np.float32); slash = np.zeros_like(vert)
    rvert = np.zeros_like(vert); rslash = np.zeros_like(vert)
    for s in range(S):
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        for h in range(Hq):
            a = OP.probe_rows(Qs[h], Ks[0], q1)
            b = OP.probe_rows(Qs[h], Ks[0], q1, OP.mixture_runs(q0, q1))
            vert[s, h, :, :q1], slash[s, h, :, :q1] = a.vert, a.slash
            rvert[s, h, :, :q1], rslash[s, h, :, :q1] = b.vert, b.slash
    idx = rs.IndexSet.for_library(p, lib_c, materialised=False)
    stats = torch.zeros((p.n_items, len(lib), 5), dtype=torch.int64, device="cuda")
    st = rs.new_status()
    t = lambda x: torch.from_numpy(x).cuda()
    rs.rs_build_indices_ranked(p, lib_c, t(vert), t(slash), t(rvert), t(rslash), None, None, None, None, idx, stats,
                               rs.new_workspace(p, lib_c), st)
    rs.check_status(st, "ranked")
    stats = stats.cpu().numpy()
    n_changed = 0
    for item in range(p.n_items):
        s, h = divmod(item, Hq)
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        for c, cand in enumerate(lib):
            if cand.pattern != PT.VERTICAL_SLASH:
                continue
            ix = PT.build_indices(cand, q0, q1, rvert[s, h][:, :q1], rslash[s, h][:, :q1], None)
            slot = item * len(lib) + c
            cnt = idx.vs_count[slot].cpu().numpy()
            assert cnt[:3].tolist() == [len(ix.V), len(ix.S), len(ix.D)]
            assert np.array_equal(idx.vs_cols[slot, :len(ix.V)].cpu().numpy(), ix.V)
            assert np.array_equal(idx.vs_offs[slot, :len(ix.S)].cpu().numpy(), ix.S)
            assert np.array_equal(idx.vs_diag[slot, :len(ix.D)].cpu().numpy(), ix.D)
            assert int(stats[item, c, 4]) == PT.pairs(ix)
            assert stats[item, c, :4].astype(np.uint64).tolist() == \
                PT.coverage_fx(ix, vert[s, h][:, :q1], slash[s, h][:, :q1]).tolist()
            plain = PT.build_indices(cand, q0, q1, vert[s, h][:, :q1], slash[s, h][:, :q1], None)
            n_changed += not np.array_equal(plain.V, ix.V)
    assert n_changed > 0                       # the mixture really picks other columns than the recent rows do


def test_layer_with_mixture_lists_runs_and_its_output_matches_the_oracle_under_its_own_lists():
    from bench import download_sets
    from oracle import attention as A
    n, Hq, Hkv = 1088, 4, 2
    L = make_layer(tiny_spec(81, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n)
    lib = [(rs.RS_VERTICAL_SLASH, 32, 48), (rs.RS_VERTICAL_SLASH, 64, 96), (rs.RS_DENSE, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=0.3, cert_max=None, mixture_lists=True), out_dtype=torch.float32)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    O = layer.forward(Q, K, V).cpu().numpy()
    rs.check_status(layer.status, "mixture lists")
    choice = layer.choice.cpu().numpy()
    cands = [PT.Candidate(*c) for c in lib]
    sets = download_sets(layer, cands, choice)
    Qs, Ks, Vs = f64_heads(L)
    mv, ms = layer._mix["vert"].cpu().numpy(), layer._mix["slash"].cpu().numpy()
    for h in range(Hq):
        if cands[choice[h]].pattern == PT.VERTICAL_SLASH:        # the lists are the top-k of the GPU's mixture masses
            ref = PT.build_indices(cands[choice[h]], 0, n, mv[0, h], ms[0, h], None)
            assert np.array_equal(sets[h].V, ref.V) and np.array_equal(sets[h].S, ref.S)
        Om, _, _ = A.masked_attention(Qs[h], Ks[h // 2], Vs[h // 2], lambda r, nk: PT.mask_rows(sets[h], r, nk))
        err = np.abs(O[h] - Om)
        assert err.max() <= 2e-2 and err.mean() <= 5e-3
