"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot compute a whole 128K layer, so: the probe, the candidate statistics, the chosen index lists and the
routing decision are checked in full for sampled heads (the oracle's probe costs O(64 n d) per head), and the attention
output is checked on sampled query blocks, each stage fed what the previous GPU stage produced.

The attention output is compared in fp32 (the library's fp32 output option) against the plain bar of 2e-2 max-abs and
5e-3 mean-abs; the bf16 output the benchmark times is then required to be the same result rounded once to bf16.
"""
import functools

import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import assert_attention_close, dev_bf16
from oracle import attention as A
from oracle import patterns as PT
from oracle import probe as OP
from oracle import routing as RT
from synth import bf16_bits_to_f64, config2_spec, config3_spec, fixed_routes_config2, make_layer
from test_gpu_pipeline import download_sets

pytestmark = pytest.mark.gpu


def _close(a, b, rtol=1e-3, floor=1e-7):
    return np.all(np.abs(a - b) <= rtol * np.abs(b) + floor)


@functools.lru_cache(maxsize=1)
def _layer(name):
    spec = {"config3": config3_spec, "config2": config2_spec}[name]()
    return spec, make_layer(spec)


def _check_rows(L, G, layer, ix, h, qb, what):
    """One 64-row query block of head h under the index set ix: fp32 output and log-sum-exp against the oracle."""
    assert layer.O.dtype == torch.float32
    Qf, Kf, Vf = (bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G]), bf16_bits_to_f64(L["V"][h // G]))
    rows = np.arange(64 * qb, 64 * qb + 64)
    Om, lo, _ = A.masked_attention(Qf, Kf, Vf, lambda r, nk: PT.mask_rows(ix, r, nk), rows, chunk=64)
    assert_attention_close(layer.O[h, 64 * qb:64 * qb + 64].cpu().numpy(), Om, what)
    assert np.abs(layer.lse_sel[h, 64 * qb:64 * qb + 64].cpu().numpy() - lo).max() < 2e-3, what


def _check_sampled_attention(L, spec, layer, sets, heads, blocks):
    G = spec.n_q_heads // spec.n_kv_heads
    for h in heads:
        for qb in blocks:
            _check_rows(L, G, layer, sets[h], h, qb, f"head {h} query block {qb}")


def _bf16_run_is_the_rounded_fp32_run(layer, Q, K, V, heads, blocks, **forward_kw):
    """The launch configuration the benchmark times writes bf16: same routes, same kernel, one rounding at the end."""
    O32, choice = layer.O, layer.choice.clone()
    layer.O = torch.empty(O32.shape, dtype=torch.bfloat16, device=O32.device)
    layer._bufs = None
    layer.forward(Q, K, V, **forward_kw)
    rs.check_status(layer.status, "bf16 output")
    assert torch.equal(layer.choice, choice)
    for h in heads:
        for qb in blocks:
            sl = slice(64 * qb, 64 * qb + 64)
            assert torch.equal(layer.O[h, sl], O32[h, sl].to(torch.bfloat16)), (h, qb)


def _assert_block_lists_match_up_to_near_ties(got_rows, want_rows, bs, qb0=0):
    """Block-sparse lists built from the fused fp32 scores against the oracle's selection on float64 scores: same
    length, ascending, diagonal kept; a block may differ only if its oracle score is a near tie of the row's k-th
    score (the smallest selected one), within the fp32 tolerance of the pooled product."""
    n_diff = 0
    for t, (got, want) in enumerate(zip(got_rows, want_rows)):
        qb = qb0 + t
        assert len(got) == len(want) and got[-1] == qb and np.all(np.diff(got) > 0), qb
        diff = np.setxor1d(got, want)
        if len(diff):
            n_diff += len(diff)
            off_diag = want[want != qb]
            kth = bs[qb, off_diag].min()
            tol = 1e-3 * max(1.0, np.abs(bs[qb, :qb + 1]).max())
            assert np.abs(bs[qb, diff] - kth).max() <= tol, (qb, diff, bs[qb, diff], kth)
    return n_diff


def test_config3_full_size_online_routing():
    spec, L = _layer("config3")
    n, Hq, Hkv = spec.n, spec.n_q_heads, spec.n_kv_heads
    p = rs.Problem(Hq, Hkv, n)
    layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(budget_frac=0.15, cert_max=0.05), out_dtype=torch.float32)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    layer.forward(Q, K, V)
    rs.check_status(layer.status, "config 3")
    cands = PT.default_library()
    assert [(c.pattern, c.b0, c.b1) for c in cands] == [tuple(c) for c in layer.cands]
    choice = layer.choice.cpu().numpy()
    stats = layer.stats.cpu().numpy()
    cov, pairs = stats[:, :, :4].astype(np.uint64), stats[:, :, 4]
    heads = [0, 9, 21, 31]
    G = Hq // Hkv
    for h in heads:
        Qf, Kf = bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G])
        pr = OP.probe_rows(Qf, Kf, n)
        vert, slash = layer.vert[0, h].cpu().numpy(), layer.slash[0, h].cpu().numpy()
        assert _close(vert, pr.vert) and _close(slash, pr.slash), h
        assert np.abs(layer.lse_probe[h, 0].cpu().numpy() - pr.lse).max() < 1e-3
        # the layer pools queries lazily: the block candidate evaluation reads (the last one) is there after the probe,
        # the others only for heads routed to block-sparse
        qp = layer.qpool[h].cpu().numpy()
        assert np.allclose(qp[-1], OP.pool_mean(Qf)[-1], rtol=1e-5, atol=1e-6)
        # candidate statistics and chosen lists from the GPU's own probe scores: bit-exact
        for c, cand in enumerate(cands):
            if cand.pattern == PT.BLOCK_SPARSE:
                assert pairs[h, c] == sum((min(cand.b0, qb + 1) - 1) * 4096 + 2080 for qb in range(n // 64))
                continue
            ix = PT.build_indices(cand, 0, n, vert, slash, None)
            assert pairs[h, c] == PT.pairs(ix), (h, cand)
            if cand.pattern != PT.DENSE:
                assert cov[h, c].tolist() == PT.coverage_fx(ix, vert, slash).tolist(), (h, cand)
            if cand.pattern == PT.VERTICAL_SLASH:
                slot = h * len(cands) + c
                cnt = layer.idx_eval.vs_count[slot].cpu().numpy()
                assert cnt[:3].tolist() == [len(ix.V), len(ix.S), len(ix.D)]
                assert np.array_equal(layer.idx_eval.vs_cols[slot, :cnt[0]].cpu().numpy(), ix.V)
                assert np.array_equal(layer.idx_eval.vs_offs[slot, :cnt[1]].cpu().numpy(), ix.S)
                assert np.array_equal(layer.idx_eval.vs_diag[slot, :cnt[2]].cpu().numpy(), ix.D)
    # routing of the whole layer from the GPU's statistics: bit-exact
    vmax = layer.vmax.cpu().numpy()
    vmax_item = np.array([vmax[0, h // G] for h in range(Hq)], np.float32)
    want, wrep = RT.route(cands, cov, 512 * pairs, vmax_item, RT.RouteParams(
        budget=int(0.15 * rs.dense_flops(p.seg_bounds, Hq)), t_probe=rs.probe_flops(p.seg_bounds, Hq), cert_max=0.05))
    assert np.array_equal(choice, want)
    rep = layer.route_report()
    assert rep["total_cost"] == wrep.total_cost and rep["n_fallback"] == wrep.n_fallback
    # attention on sampled query blocks under the routed masks
    sets = download_sets(layer, cands, choice)
    _check_sampled_attention(L, spec, layer, sets, heads, [3, 1021, 2047])
    # kernel-side mass on the probe rows equals builder-side coverage
    m_rows = layer.m_row.cpu().numpy()
    for h in heads:
        if cands[choice[h]].pattern != PT.DENSE:
            m_hat, _ = PT.m_hat_from_fx(cov[h, choice[h]])
            assert abs(m_rows[h].mean() - m_hat) < 2e-3
    _bf16_run_is_the_rounded_fp32_run(layer, Q, K, V, heads, [3, 1021, 2047])


def test_config2_full_size_fixed_routes():
    spec, L = _layer("config2")
    n, Hq, Hkv = spec.n, spec.n_q_heads, spec.n_kv_heads
    p = rs.Problem(Hq, Hkv, n)
    lib = [(1, 128, 1024), (2, 1000, 6096), (3, 100, 0), (0, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=1.0, cert_max=None), out_dtype=torch.float32)
    pat = fixed_routes_config2(Hq)
    fixed = np.array([{1: 0, 2: 1, 3: 2, 0: 3}[int(x)] for x in pat], dtype=np.int32)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    layer.forward(Q, K, V, fixed_choice=torch.from_numpy(fixed).cuda())
    rs.check_status(layer.status, "config 2")
    cands = [PT.Candidate(*c) for c in lib]
    sets = download_sets(layer, cands, fixed)
    heads = [int(np.where(pat == k)[0][0]) for k in (1, 2, 3, 0)]        # one head of every pattern
    # the materialised vertical-slash / block-sparse lists equal the oracle's selection on the GPU's scores
    G = Hq // Hkv
    for h in heads:
        if cands[fixed[h]].pattern == PT.VERTICAL_SLASH:
            ref = PT.build_indices(cands[fixed[h]], 0, n, layer.vert[0, h].cpu().numpy(), layer.slash[0, h].cpu().numpy())
            assert np.array_equal(sets[h].V, ref.V) and np.array_equal(sets[h].S, ref.S) and np.array_equal(sets[h].D, ref.D)
        if cands[fixed[h]].pattern == PT.BLOCK_SPARSE:
            bs = OP.block_scores(bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G]), 0, n)
            ref = PT.build_block_sparse(bs, 100, 0, n // 64)
            n_diff = _assert_block_lists_match_up_to_near_ties(sets[h].blk, ref, bs)
            assert n_diff <= 0.002 * 100 * (n // 64)          # and near ties are rare
    _check_sampled_attention(L, spec, layer, sets, heads, [1, 255, 511])
    _bf16_run_is_the_rounded_fp32_run(layer, Q, K, V, heads, [1, 255, 511], fixed_choice=torch.from_numpy(fixed).cuda())


def test_block_sparse_at_128k_fixed_routes():
    """The block-sparse family at n = 131072 (2048 key blocks per row; Section 3.1): heads fixed to block-sparse with
    k_b = 100 and k_b = 400, one vertical-slash and one dense head, the rest A-shape.  Every block list of two block-sparse
    heads against the oracle's selection (near ties of the fused fp32 scores allowed, and only those), and the
    attention output on sampled query blocks under the GPU's own lists."""
    spec, L = _layer("config3")
    n, Hq, Hkv = spec.n, spec.n_q_heads, spec.n_kv_heads
    p = rs.Problem(Hq, Hkv, n)
    lib = [(3, 100, 0), (3, 400, 0), (2, 1000, 6096), (1, 128, 1024), (0, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=1.0, cert_max=None), out_dtype=torch.float32)
    fixed = np.full(Hq, 3, dtype=np.int32)
    fixed[[2, 13, 22]] = 0          # k_b = 100
    fixed[[5, 18, 31]] = 1          # k_b = 400
    fixed[9], fixed[27] = 2, 4
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    fc = torch.from_numpy(fixed).cuda()
    layer.forward(Q, K, V, fixed_choice=fc)
    rs.check_status(layer.status, "block-sparse at 128K")
    cands = [PT.Candidate(*c) for c in lib]
    sets = download_sets(layer, cands, fixed)
    G, nb = Hq // Hkv, n // 64
    for h in (13, 31):
        bs = OP.block_scores(bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G]), 0, n)
        k_b = cands[fixed[h]].b0
        ref = PT.build_block_sparse(bs, k_b, 0, nb)
        n_diff = _assert_block_lists_match_up_to_near_ties(sets[h].blk, ref, bs)
        assert n_diff <= 0.002 * k_b * nb
    heads, blocks = [13, 31, 2, 9], [0, 77, 1021, 2047]
    _check_sampled_attention(L, spec, layer, sets, heads, blocks)
    _bf16_run_is_the_rounded_fp32_run(layer, Q, K, V, heads, blocks, fixed_choice=fc)


def test_config4_full_size_segmented_layer():
    """One layer of the segmented 128K recipe (four segments of 32K with different planted structure, per-segment
    routing, one launch): probe and candidate statistics of sampled (segment, head) items, the routing of all 128 items,
    and the attention output on sampled query blocks of every segment (first, interior and last block)."""
    from synth import config4_layer_spec
    spec = config4_layer_spec(0, n=131072, seg_len=32768)
    L = make_layer(spec)
    n, Hq, Hkv = spec.n, spec.n_q_heads, spec.n_kv_heads
    bounds = spec.seg_bounds()
    p = rs.Problem(Hq, Hkv, n, bounds)
    layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(budget_frac=0.15, cert_max=0.05), out_dtype=torch.float32)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    layer.forward(Q, K, V)
    rs.check_status(layer.status, "config 4")
    cands = PT.default_library()
    choice = layer.choice.cpu().numpy()
    stats = layer.stats.cpu().numpy()
    cov, pairs = stats[:, :, :4].astype(np.uint64), stats[:, :, 4]
    G = Hq // Hkv
    sampled = [(0, 3), (1, 12), (2, 22), (3, 31)]                     # (segment, head)
    for s, h in sampled:
        q0, q1 = bounds[s], bounds[s + 1]
        item = s * Hq + h
        Qf, Kf = bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G])
        pr = OP.probe_rows(Qf, Kf, q1)
        vert, slash = layer.vert[s, h].cpu().numpy(), layer.slash[s, h].cpu().numpy()
        assert _close(vert[:, :q1], pr.vert) and _close(slash[:, :q1], pr.slash), (s, h)
        assert np.all(vert[:, q1:] == 0)
        assert np.abs(layer.lse_probe[h, s].cpu().numpy() - pr.lse).max() < 1e-3
        for c, cand in enumerate(cands):
            if cand.pattern == PT.BLOCK_SPARSE:
                assert pairs[item, c] == sum((min(cand.b0, qb + 1) - 1) * 4096 + 2080 for qb in range(q0 // 64, q1 // 64))
                continue
            ix = PT.build_indices(cand, q0, q1, vert[:, :q1], slash[:, :q1], None)
            assert pairs[item, c] == PT.pairs(ix), (s, h, cand)
            if cand.pattern != PT.DENSE:
                assert cov[item, c].tolist() == PT.coverage_fx(ix, vert[:, :q1], slash[:, :q1]).tolist(), (s, h, cand)
    vmax = layer.vmax.cpu().numpy()
    vmax_item = np.array([vmax[it // Hq, (it % Hq) // G] for it in range(p.n_items)], np.float32)
    want, wrep = RT.route(cands, cov, 512 * pairs, vmax_item, RT.RouteParams(
        budget=int(0.15 * rs.dense_flops(p.seg_bounds, Hq)), t_probe=rs.probe_flops(p.seg_bounds, Hq), cert_max=0.05))
    assert np.array_equal(choice, want)
    rep = layer.route_report()
    assert rep["total_cost"] == wrep.total_cost and rep["n_fallback"] == wrep.n_fallback
    assert len(set(choice.tolist())) > 2                              # the segments really get different routes
    sets = download_sets(layer, cands, choice)
    for s, h in sampled:
        q0, q1 = bounds[s], bounds[s + 1]
        for qb in (q0 // 64, (q0 + q1) // 128 + 1, q1 // 64 - 1):
            _check_rows(L, G, layer, sets[s * Hq + h], h, qb, f"segment {s} head {h} query block {qb}")
