"""Pins for the oracle's pattern library (Section 3.1): index sets, masks, pair counts, coverage. CPU only."""
import numpy as np
import pytest

from oracle import attention as A
from oracle import patterns as PT
from oracle import probe as P
from synth import bf16_bits_to_f64, make_layer, tiny_spec

C = PT.Candidate


def _head(seed=3, n=512):
    L = make_layer(tiny_spec(seed, n, 1, 1))
    return (bf16_bits_to_f64(L["Q"][0]), bf16_bits_to_f64(L["K"][0]), bf16_bits_to_f64(L["V"][0]))


def _probe(seed=3, n=512, q0=0, q1=None):
    Q, K, V = _head(seed, n)
    q1 = n if q1 is None else q1
    pr = P.probe_rows(Q, K, q1)
    bs = P.block_scores(Q, K, q0, q1)
    return Q, K, V, pr, bs


CANDS = [C(PT.DENSE), C(PT.A_SHAPE, 8, 96), C(PT.A_SHAPE, 70, 130), C(PT.VERTICAL_SLASH, 24, 40),
         C(PT.VERTICAL_SLASH, 5, 3), C(PT.VERTICAL_SLASH, 24, 40, strict=True), C(PT.BLOCK_SPARSE, 3), C(PT.BLOCK_SPARSE, 1)]


def test_fx_and_topk_order():
    assert int(PT.fx(np.float32(0.5))) == 1 << 31 and int(PT.fx(np.float32(16.0))) == 16 << 32
    assert int(PT.fx(np.float32(1e-12))) == 0
    keys = np.array([5, 9, 9, 1, 9, 5], dtype=np.uint64)
    assert PT.topk_desc(keys, 4).tolist() == [1, 2, 4, 0]          # key descending, ties by lower index
    assert PT.topk_desc(np.array([0.0, -0.0, 1.0, 1.0], np.float32), 3).tolist() == [2, 3, 0]
    assert PT.topk_desc(keys, 99).tolist() == [1, 2, 4, 0, 5, 3]    # k clamps


def test_block_diagonals_touched_by_a_slash_brute_force():
    for o in range(0, 400, 7):
        touched = set()
        for qb in range(8):
            for i in range(64 * qb, 64 * qb + 64):
                if i - o >= 0:
                    touched.add(qb - (i - o) // 64)
        want = {o // 64, (o + 63) // 64}
        assert touched <= want and (o >= 512 or touched == {x for x in want if x < 8})


def test_lists_are_sorted_unique_in_range():
    _, _, _, pr, bs = _probe(n=512)
    V, S, D = PT.build_vertical_slash(pr.vert, pr.slash, 24, 40, 512)
    for a, k, hi in ((V, 24, 512), (S, 40, 512), (D, None, 8)):
        assert np.all(np.diff(a) > 0) and a.min() >= 0 and a.max() < hi
        assert k is None or len(a) == k
    assert S[0] == 0
    assert set(D) == {x for o in S for x in (o // 64, (o + 63) // 64) if x < 8}
    blk = PT.build_block_sparse(bs, 3, 0, 8)
    for qb, sel in enumerate(blk):
        assert np.all(np.diff(sel) > 0) and sel[-1] == qb and len(sel) == min(3, qb + 1)


def test_topk_selects_the_largest_mass():
    _, _, _, pr, _ = _probe(seed=8, n=512)
    V, S, _ = PT.build_vertical_slash(pr.vert, pr.slash, 10, 6, 512)
    kv = PT.line_keys(pr.vert)
    assert kv[V].min() >= np.delete(kv, V).max()
    ks = PT.line_keys(pr.slash)
    rest = np.setdiff1d(np.arange(1, 512), S)
    assert ks[S[1:]].min() >= ks[rest].max()


def test_a_shape_is_data_independent_and_token_granular():
    ix = PT.build_indices(C(PT.A_SHAPE, 5, 10), 0, 128)
    M = PT.explicit_mask(ix, 128)
    assert M[100, 4] and not M[100, 5] and M[100, 91] and not M[100, 90] and M[100, 100] and not M[100, 101]


@pytest.mark.parametrize("q0,q1", [(0, 512), (256, 512), (128, 384)])
def test_pairs_closed_form_equals_explicit_mask(q0, q1):
    _, _, _, pr, bs = _probe(seed=5, n=512, q0=q0, q1=q1)
    for cand in CANDS:
        if cand.strict:
            continue
        ix = PT.build_indices(cand, q0, q1, pr.vert, pr.slash, bs)
        assert PT.pairs(ix) == int(PT.explicit_mask(ix, 512).sum()), cand


def test_every_pattern_keeps_the_diagonal():
    _, _, _, pr, bs = _probe(seed=6, n=384)
    for cand in CANDS:
        M = PT.explicit_mask(PT.build_indices(cand, 0, 384, pr.vert, pr.slash, bs), 384)
        assert M[np.arange(384), np.arange(384)].all(), cand


@pytest.mark.parametrize("q0,q1", [(0, 512), (192, 448)])
def test_coverage_fx_matches_plain_definition(q0, q1):
    _, _, _, pr, bs = _probe(seed=7, n=512, q0=q0, q1=q1)
    for cand in CANDS:
        if cand.pattern == PT.DENSE:
            continue
        ix = PT.build_indices(cand, q0, q1, pr.vert, pr.slash, bs)
        plain = PT.coverage_plain(ix, pr.P)
        assert np.all(plain <= 1 + 1e-12)
        if cand.strict:
            continue
        cov = PT.coverage_fx(ix, pr.vert, pr.slash)
        assert np.allclose(cov.astype(np.float64) / (16 * 2.0 ** 32), plain, atol=1e-6), cand
        m_hat, u = PT.m_hat_from_fx(cov)
        assert abs(m_hat - plain.mean()) < 1e-6 and abs(u - (plain.max() - plain.min())) < 1e-6


def test_a_shape_overlap_cases():
    _, _, _, pr, _ = _probe(seed=7, n=512)
    full = PT.coverage_fx(PT.build_indices(C(PT.A_SHAPE, 8, 600), 0, 512), pr.vert, pr.slash)
    assert np.allclose(full.astype(float) / (16 * 2.0 ** 32), 1.0, atol=1e-6)
    with pytest.raises(ValueError):
        PT.coverage_fx(PT.build_indices(C(PT.A_SHAPE, 100, 400), 0, 512), pr.vert, pr.slash)


def test_strict_is_a_subset_of_block_and_budgets_nest():
    _, _, _, pr, bs = _probe(seed=9, n=512)
    strict = PT.build_indices(C(PT.VERTICAL_SLASH, 24, 40, strict=True), 0, 512, pr.vert, pr.slash)
    block = PT.build_indices(C(PT.VERTICAL_SLASH, 24, 40), 0, 512, pr.vert, pr.slash)
    Ms, Mb = PT.explicit_mask(strict, 512), PT.explicit_mask(block, 512)
    assert not (Ms & ~Mb).any() and Ms.sum() < Mb.sum()
    assert PT.coverage_plain(strict, pr.P).mean() <= PT.coverage_plain(block, pr.P).mean() + 1e-12
    small = PT.build_indices(C(PT.VERTICAL_SLASH, 10, 12), 0, 512, pr.vert, pr.slash)
    assert set(small.V) <= set(block.V) and set(small.S) <= set(block.S) and set(small.D) <= set(block.D)
    b2 = PT.build_block_sparse(bs, 2, 0, 8)
    b4 = PT.build_block_sparse(bs, 4, 0, 8)
    assert all(set(a) <= set(b) for a, b in zip(b2, b4))


def test_budget_at_least_n_gives_the_causal_mask():
    _, _, _, pr, bs = _probe(seed=10, n=256)
    causal = np.tril(np.ones((256, 256), bool))
    for cand in (C(PT.VERTICAL_SLASH, 256, 1), C(PT.VERTICAL_SLASH, 1, 256), C(PT.BLOCK_SPARSE, 4),
                 C(PT.A_SHAPE, 0, 256), C(PT.VERTICAL_SLASH, 999, 999, strict=True)):
        ix = PT.build_indices(cand, 0, 256, pr.vert, pr.slash, bs)
        assert np.array_equal(PT.explicit_mask(ix, 256), causal), cand
        assert abs(PT.coverage_plain(ix, pr.P).mean() - 1) < 1e-12
    ix = PT.build_indices(C(PT.BLOCK_SPARSE, 4), 0, 256, pr.vert, pr.slash, bs)
    assert abs(PT.m_hat_from_fx(PT.coverage_fx(ix, pr.vert, pr.slash))[0] - 1) < 256 * 2.0 ** -32 * 4


def test_block_sparse_picks_the_best_pooled_scores():
    _, _, _, _, bs = _probe(seed=11, n=512)
    blk = PT.build_block_sparse(bs, 3, 0, 8)
    for qb in range(3, 8):
        others = np.setdiff1d(np.arange(qb), blk[qb])
        assert bs[qb, blk[qb][:-1]].min() >= bs[qb, others].max()


def test_masked_attention_under_each_pattern_matches_explicit_mask():
    Q, K, V, pr, bs = _probe(seed=12, n=256)
    for cand in CANDS:
        ix = PT.build_indices(cand, 0, 256, pr.vert, pr.slash, bs)
        M = PT.explicit_mask(ix, 256)
        O1, l1, _ = A.masked_attention(Q, K, V, lambda r, nk: PT.mask_rows(ix, r, nk))
        O2, l2, _ = A.masked_attention(Q, K, V, lambda r, nk: M[r][:, :nk])
        assert np.array_equal(O1, O2) and np.array_equal(l1, l2)


def test_default_library_shape():
    lib = PT.default_library()
    assert len(lib) == 13 and lib[-1].pattern == PT.DENSE
    assert [c.pattern for c in lib].count(PT.VERTICAL_SLASH) == 4


def test_mixture_coverage_closed_cases():
    """Coverage of mask rows at the pooled probe's block resolution: dense collects everything, a window that ends on
    block boundaries collects exactly its blocks, a half-covered block collects half of its mass."""
    from oracle.patterns import A_SHAPE, DENSE, VERTICAL_SLASH, Candidate, build_indices, fx, mixture_coverage_fx, mixture_u
    n = 512
    a = np.zeros(n // 64, dtype=np.float32)
    a[:] = [0.25, 0.03125, 0.125, 0.0625, 0.03125, 0.125, 0.125, 0.25]
    i = 447                                                         # last row of block 6: blocks 0..6 fully visible
    dense = build_indices(Candidate(DENSE), 0, n)
    assert mixture_coverage_fx(dense, a, i, n) == int(fx(a[:7]).sum())
    win = build_indices(Candidate(A_SHAPE, 64, 128), 0, n)          # sink = block 0, window = keys 320..447 = blocks 5, 6
    assert mixture_coverage_fx(win, a, i, n) == int(fx(a[[0, 5, 6]]).sum())
    half = build_indices(Candidate(A_SHAPE, 32, 96), 0, n)          # half of block 0, keys 352..447 = half of block 5 + block 6
    assert mixture_coverage_fx(half, a, i, n) == int(fx(a[0])) * 32 // 64 + int(fx(a[5])) * 32 // 64 + int(fx(a[6]))
    # a row in the middle of a block: window = keys 74..201 = 54 keys of block 1, block 2, the 10 visible keys of block 3
    i2 = 64 * 3 + 9
    assert mixture_coverage_fx(win, a, i2, n) == int(fx(a[0])) + int(fx(a[1])) * 54 // 64 + int(fx(a[2])) + int(fx(a[3]))
    # vertical-slash: columns count individually, block diagonals cover whole blocks
    from oracle.patterns import IndexSet
    vs = IndexSet(cand=Candidate(VERTICAL_SLASH, 2, 2), q0=0, q1=n, V=np.array([70, 71]), S=np.array([0, 1]),
                  D=np.array([0, 1]))                           # two columns in block 1, block diagonals 0 and 1
    assert mixture_coverage_fx(vs, a, i, n) == int(fx(a[1])) * 2 // 64 + int(fx(a[5])) + int(fx(a[6]))
    assert abs(mixture_u(np.array([2 ** 32 * 16, 2 ** 32 * 8, 2 ** 32 * 12, 0], dtype=np.uint64), [32, 16, 16, 0]) - 0.25) < 1e-15
