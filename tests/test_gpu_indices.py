"""GPU parity: rs_build_indices against the oracle, bit-exact when fed the oracle's probe scores."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import c_library, f64_heads, oracle_probe_all
from oracle import patterns as PT
from oracle import probe as OP
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu
C = PT.Candidate

LIB = [C(PT.A_SHAPE, 8, 64), C(PT.A_SHAPE, 8, 128), C(PT.VERTICAL_SLASH, 16, 24), C(PT.VERTICAL_SLASH, 40, 70),
       C(PT.VERTICAL_SLASH, 5000, 1), C(PT.BLOCK_SPARSE, 2), C(PT.BLOCK_SPARSE, 5), C(PT.DENSE)]


def oracle_scores(L, p):
    Qs, Ks, _ = f64_heads(L)
    probes = oracle_probe_all(Qs, Ks, p)
    S, Hq, n, nb = p.n_segments, p.n_q_heads, p.n_keys, p.n_keys // 64
    vert = np.zeros((S, Hq, 4, n), np.float32)
    slash = np.zeros((S, Hq, 4, n), np.float32)
    bscore = np.zeros((p.n_items, nb, nb), np.float32)
    for item, (pr, bs) in probes.items():
        s, h = divmod(item, Hq)
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        vert[s, h, :, :q1] = pr.vert
        slash[s, h, :, :q1] = pr.slash
        bscore[item, q0 // 64:q1 // 64, :q1 // 64] = np.where(np.isfinite(bs), bs, 0)
    return probes, vert, slash, bscore


def gpu_build(p, lib_c, vert, slash, bscore, qpool, kpool, choice, want_stats=True):
    idx = rs.IndexSet.for_library(p, lib_c, materialised=choice is not None)
    stats = torch.zeros((p.n_items, len(lib_c), 5), dtype=torch.int64, device="cuda") if want_stats else None
    ws = rs.new_workspace(p, lib_c)
    st = rs.new_status()
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    ch = None if choice is None else torch.tensor(choice, dtype=torch.int32, device="cuda")
    rs.rs_build_indices(p, lib_c, t(vert), t(slash), t(qpool), t(kpool), t(bscore), ch, idx, stats, ws, st)
    rs.check_status(st, "build_indices")
    return idx, (None if stats is None else stats.cpu().numpy())


def check_slot_vs(idx, slot, ix):
    cnt = idx.vs_count[slot].cpu().numpy()
    assert cnt[:3].tolist() == [len(ix.V), len(ix.S), len(ix.D)], (slot, cnt, len(ix.V), len(ix.S), len(ix.D))
    assert np.array_equal(idx.vs_cols[slot, :len(ix.V)].cpu().numpy(), ix.V)
    assert np.array_equal(idx.vs_offs[slot, :len(ix.S)].cpu().numpy(), ix.S)
    assert np.array_equal(idx.vs_diag[slot, :len(ix.D)].cpu().numpy(), ix.D)


# libraries without one of the families: the kernels that serve two families in one launch then run with one kind of block
LIB_NO_VS = [C(PT.A_SHAPE, 8, 64), C(PT.BLOCK_SPARSE, 3), C(PT.BLOCK_SPARSE, 7), C(PT.DENSE)]
LIB_NO_BS = [C(PT.VERTICAL_SLASH, 16, 24), C(PT.A_SHAPE, 8, 128), C(PT.VERTICAL_SLASH, 40, 70), C(PT.DENSE)]


@pytest.mark.parametrize("n,Hq,Hkv,bounds,LIB", [(832, 4, 2, None, LIB), (1344, 2, 1, [0, 448, 1344], LIB),
                                                 (1344, 2, 1, [0, 448, 1344], LIB_NO_VS), (832, 4, 2, None, LIB_NO_BS)])
def test_evaluation_mode_is_bit_exact(n, Hq, Hkv, bounds, LIB):
    L = make_layer(tiny_spec(41 + n, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, bounds or [0, n])
    probes, vert, slash, bscore = oracle_scores(L, p)
    lib_c = c_library(LIB)
    idx, stats = gpu_build(p, lib_c, vert, slash, bscore, None, None, None)
    for item in range(p.n_items):
        s = item // Hq
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        pr, bs = probes[item]
        for c, cand in enumerate(LIB):
            slot = item * len(LIB) + c
            ix = PT.build_indices(cand, q0, q1, pr.vert, pr.slash, bs)
            assert int(stats[item, c, 4]) == PT.pairs(ix), (item, cand)
            if cand.pattern == PT.DENSE:
                continue
            assert stats[item, c, :4].astype(np.uint64).tolist() == PT.coverage_fx(ix, pr.vert, pr.slash).tolist(), (item, cand)
            if cand.pattern == PT.VERTICAL_SLASH:
                check_slot_vs(idx, slot, ix)
            if cand.pattern == PT.BLOCK_SPARSE:
                want = ix.blk[-1]
                assert int(idx.bs_count[slot]) == len(want)
                assert np.array_equal(idx.bs_blk[slot, :len(want)].cpu().numpy(), want)


def test_materialise_mode_is_bit_exact_and_ties_are_broken_by_index():
    n, Hq, Hkv = 1024, 4, 2
    L = make_layer(tiny_spec(43, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, [0, 384, 1024])
    probes, vert, slash, bscore = oracle_scores(L, p)
    # plant exact ties: equal masses on a run of columns / offsets and equal block scores
    vert[:, :, :, 100:140] = 0.25
    slash[:, :, :, 50:90] = 0.125
    bscore[:, :, 2:6] = 0.5
    lib_c = c_library(LIB)
    choice = [(3 * item + 2) % len(LIB) for item in range(p.n_items)]
    idx, stats = gpu_build(p, lib_c, vert, slash, bscore, None, None, choice)
    nb = n // 64
    for item in range(p.n_items):
        s, h = divmod(item, Hq)
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        cand = LIB[choice[item]]
        bs = np.where(np.arange(nb)[None, :] <= np.arange(q0 // 64, q1 // 64)[:, None], bscore[item, q0 // 64:q1 // 64], -np.inf)
        ix = PT.build_indices(cand, q0, q1, vert[s, h][:, :q1], slash[s, h][:, :q1], bs)
        assert int(stats[item, choice[item], 4]) == PT.pairs(ix)
        if cand.pattern == PT.VERTICAL_SLASH:
            check_slot_vs(idx, item, ix)
        if cand.pattern == PT.BLOCK_SPARSE:
            for t, sel in enumerate(ix.blk):
                row = h * nb + q0 // 64 + t
                assert int(idx.bs_count[row]) == len(sel)
                assert np.array_equal(idx.bs_blk[row, :len(sel)].cpu().numpy(), sel), (item, t)


def test_fused_block_scores_select_the_same_blocks_up_to_near_ties():
    n, Hq, Hkv = 1536, 2, 1
    L = make_layer(tiny_spec(47, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n)
    Qs, Ks, _ = f64_heads(L)
    probes, vert, slash, bscore = oracle_scores(L, p)
    qpool = np.stack([OP.pool_mean(q) for q in Qs]).astype(np.float32)
    kpool = np.stack([OP.pool_mean(k) for k in Ks]).astype(np.float32)
    lib = [C(PT.BLOCK_SPARSE, 6), C(PT.DENSE)]
    lib_c = c_library(lib)
    idx, _ = gpu_build(p, lib_c, vert, slash, None, qpool, kpool, [0, 0], want_stats=False)
    nb = n // 64
    for h in range(Hq):
        bs = probes[h][1]
        want = PT.build_block_sparse(bs, 6, 0, nb)
        for qb in range(nb):
            got = idx.bs_blk[h * nb + qb, :int(idx.bs_count[h * nb + qb])].cpu().numpy()
            assert len(got) == len(want[qb]) and got[-1] == qb and np.all(np.diff(got) > 0)
            diff = np.setxor1d(got, want[qb])
            if len(diff):      # only blocks whose scores are within the fp32 tolerance of each other may swap
                sc = bs[qb, diff]
                assert sc.max() - sc.min() <= 1e-3 * max(1.0, np.abs(bs[qb, :qb + 1]).max())
    # evaluation mode from the pooled arrays (no vertical-slash candidate: the statistics kernel and the evaluation
    # kernel run with their block-sparse parts only): the list of the last query block is the materialised row
    idx_e, stats = gpu_build(p, lib_c, vert, slash, None, qpool, kpool, None)
    for h in range(Hq):
        row = h * nb + nb - 1
        got_m = idx.bs_blk[row, :int(idx.bs_count[row])].cpu().numpy()
        slot = h * len(lib)
        got_e = idx_e.bs_blk[slot, :int(idx_e.bs_count[slot])].cpu().numpy()
        assert np.array_equal(got_e, got_m)
        ix = PT.IndexSet(cand=lib[0], q0=0, q1=n)
        ix.blk = [None] * (nb - 1) + [got_e]
        assert stats[h, 0, :4].astype(np.uint64).tolist() == PT.coverage_fx(ix, probes[h][0].vert, probes[h][0].slash).tolist()


def test_argument_checks():
    p = rs.Problem(2, 1, 256)
    lib_c = c_library([C(PT.A_SHAPE, 100, 150), C(PT.DENSE)])    # sink and window overlap on the probe rows
    z = np.zeros((1, 2, 4, 256), np.float32)
    with pytest.raises(rs.RouteSparseError):
        gpu_build(p, lib_c, z, z, None, None, None, None)
