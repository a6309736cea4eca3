"""GPU parity: coverage of the candidates on the rows of the query mixture (rs_mixture_coverage) and the router fed
with the resulting subset disagreement, bit-exact against the oracle when both read the GPU's pooled-probe
probabilities and index lists."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import dev_bf16
from oracle import patterns as PT
from oracle import routing as RT
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu

LIB = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_A_SHAPE, 16, 200), (rs.RS_VERTICAL_SLASH, 48, 160), (rs.RS_VERTICAL_SLASH, 96, 320),
       (rs.RS_BLOCK_SPARSE, 3, 0), (rs.RS_BLOCK_SPARSE, 6, 0), (rs.RS_DENSE, 0, 0)]
CANDS = [PT.Candidate(c[0], c[1], c[2]) for c in LIB]


def bs_lists_for_all_blocks(layer, Q, K, V, c):
    """The block lists the materialising kernel writes when every head is routed to block-sparse candidate c."""
    layer.choice.fill_(c)
    layer.materialise()
    torch.cuda.synchronize()
    return layer.idx.bs_blk.cpu().numpy().copy(), layer.idx.bs_count.cpu().numpy().copy()


@pytest.mark.parametrize("n,Hq,Hkv,bounds", [(1024, 4, 2, None), (1216, 2, 1, [0, 448, 1216])])
def test_mixture_coverage_and_router(n, Hq, Hkv, bounds):
    L = make_layer(tiny_spec(61 + n, n, Hq, Hkv))
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
    layer = rs.RoutedPrefillLayer(p, LIB, rs.RouteConfig(budget_frac=0.35, cert_max=None, mixture_u=True))
    layer.probe(Q, K, V)
    layer.evaluate_candidates()
    layer.mixture_coverage(Q, K)
    torch.cuda.synchronize()
    rs.check_status(layer.status, "mixture coverage")
    got = layer.covmix.cpu().numpy().astype(np.uint64)
    A = layer.pp["A"].cpu().numpy()
    rows = layer.pp["rows"].cpu().numpy()
    sub = layer.pp["sub"]
    ev = layer.idx_eval
    cnt = ev.vs_count.cpu().numpy()
    cols, offs, diag = (t.cpu().numpy() for t in (ev.vs_cols, ev.vs_offs, ev.vs_diag))
    nb = n // 64
    bs = {c: bs_lists_for_all_blocks(layer, Q, K, V, c) for c, cd in enumerate(LIB) if cd[0] == rs.RS_BLOCK_SPARSE}
    want = np.zeros_like(got)
    for item in range(p.n_items):
        s, h = divmod(item, Hq)
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        for c, cand in enumerate(CANDS):
            ix = PT.IndexSet(cand=cand, q0=q0, q1=q1)
            if cand.pattern == PT.VERTICAL_SLASH:
                sl = item * len(LIB) + c
                ix.V, ix.S, ix.D = cols[sl, :cnt[sl, 0]], offs[sl, :cnt[sl, 1]], diag[sl, :cnt[sl, 2]]
            elif cand.pattern == PT.BLOCK_SPARSE:
                blk, bcnt = bs[c]
                ix.blk = [blk[h * nb + qb, :bcnt[h * nb + qb]] for qb in range(q0 // 64, q1 // 64)]
            for t in range(rows.shape[1]):
                b = max(k for k in range(len(sub) - 1) if t >= sub[k])
                want[item, c, b] += np.uint64(PT.mixture_coverage_fx(ix, A[s, h, t], int(rows[s, t]), n))
    assert np.array_equal(got, want)
    # dense collects (almost) everything: the fp32 probabilities of a row sum to 1 within rounding
    dense_c = len(LIB) - 1
    per_row = got[:, dense_c, :3].astype(np.float64) / (np.array([32, 16, 16]) * 2.0 ** 32)
    assert np.all(np.abs(per_row - 1.0) < 1e-5)

    # the router with u = disagreement among the subsets
    layer.route()
    torch.cuda.synchronize()
    choice = layer.choice.cpu().numpy()
    stats = layer.stats.cpu().numpy()
    cov = stats[:, :, :4].astype(np.uint64); pairs = stats[:, :, 4]
    u_mix = np.array([[PT.mixture_u(got[it, c], [32, 16, 16, 0]) for c in range(len(LIB))] for it in range(p.n_items)])
    vm = layer.vmax.cpu().numpy()
    vmax_item = np.array([vm[it // Hq, (it % Hq) // (Hq // Hkv)] for it in range(p.n_items)], np.float32)
    prm = RT.RouteParams(budget=int(0.35 * rs.dense_flops(p.seg_bounds, Hq)), t_probe=rs.probe_flops(p.seg_bounds, Hq),
                         alpha=1.0, cert_max=None, u_mix=u_mix)
    want_choice, _ = RT.route(CANDS, cov, 512 * pairs, vmax_item, prm)
    assert np.array_equal(choice, want_choice)
    # and the subsets do disagree somewhere on this layer, so the term is not idle
    assert float(u_mix[:, :dense_c].max()) > 0.01
