"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot compute a whole 128K layer, so: the probe, the candidate statistics, the chosen index lists and the
routing decision are checked in full for sampled heads (the oracle's probe costs O(64 n d) per head), and the attention
output is checked on sampled query blocks, each stage fed what the previous GPU stage produced.
"""
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


def _check_sampled_attention(L, spec, layer, sets, heads, blocks):
    G = spec.n_q_heads // spec.n_kv_heads
    O = layer.O
    for h in heads:
        Qf, Kf, Vf = (bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G]), bf16_bits_to_f64(L["V"][h // G]))
        ix = sets[h]
        for qb in blocks:
            rows = np.arange(64 * qb, 64 * qb + 64)
            Om, lo, _ = A.masked_attention(Qf, Kf, Vf, lambda r, nk: PT.mask_rows(ix, r, nk), rows, chunk=64)
            got = O[h, 64 * qb:64 * qb + 64].float().cpu().numpy()
            err = np.abs(got - Om)
            # bf16 output: add half an ulp of the largest output to the max-abs bar
            assert err.max() <= 2e-2 + 2.0 ** -9 * np.abs(Om).max() and err.mean() <= 5e-3, (h, qb, err.max())
            assert np.abs(layer.lse_sel[h, 64 * qb:64 * qb + 64].cpu().numpy() - lo).max() < 2e-3


def test_config3_full_size_online_routing():
    spec = config3_spec(131072)
    L = make_layer(spec)
    n, Hq, Hkv = spec.n, spec.n_q_heads, spec.n_kv_heads
    p = rs.Problem(Hq, Hkv, n)
    layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(budget_frac=0.15, cert_max=0.05))
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


def test_config2_full_size_fixed_routes():
    spec = config2_spec(32768)
    L = make_layer(spec)
    n, Hq, Hkv = spec.n, spec.n_q_heads, spec.n_kv_heads
    p = rs.Problem(Hq, Hkv, n)
    lib = [(1, 128, 1024), (2, 1000, 6096), (3, 100, 0), (0, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=1.0, cert_max=None))
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
            n_diff = sum(len(np.setxor1d(a, b)) for a, b in zip(sets[h].blk, ref))
            assert n_diff <= 0.002 * 100 * (n // 64)          # only near-ties of the fp32 fused scores may differ
    _check_sampled_attention(L, spec, layer, sets, heads, [1, 255, 511])


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
    layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(budget_frac=0.15, cert_max=0.05))
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
    O = layer.O
    for s, h in sampled:
        q0, q1 = bounds[s], bounds[s + 1]
        ix = sets[s * Hq + h]
        Qf, Kf, Vf = (bf16_bits_to_f64(L["Q"][h]), bf16_bits_to_f64(L["K"][h // G]), bf16_bits_to_f64(L["V"][h // G]))
        for qb in (q0 // 64, (q0 + q1) // 128 + 1, q1 // 64 - 1):
            rows = np.arange(64 * qb, 64 * qb + 64)
            Om, lo, _ = A.masked_attention(Qf, Kf, Vf, lambda r, nk: PT.mask_rows(ix, r, nk), rows, chunk=64)
            got = O[h, 64 * qb:64 * qb + 64].float().cpu().numpy()
            err = np.abs(got - Om)
            assert err.max() <= 2e-2 + 2.0 ** -9 * np.abs(Om).max() and err.mean() <= 5e-3, (s, h, qb, err.max())
            assert np.abs(layer.lse_sel[h, 64 * qb:64 * qb + 64].cpu().numpy() - lo).max() < 2e-3
