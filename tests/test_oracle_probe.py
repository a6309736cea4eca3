"""Pins for the oracle's probe (Eq. 3 in the last-64-query form). CPU only."""
import numpy as np

from oracle import attention as A
from oracle import probe as P
from synth import bf16_bits_to_f64, make_layer, tiny_spec


def _head(seed=3, n=512):
    L = make_layer(tiny_spec(seed, n, 1, 1))
    return (bf16_bits_to_f64(L["Q"][0]), bf16_bits_to_f64(L["K"][0]), bf16_bits_to_f64(L["V"][0]))


def test_masses_sum_to_number_of_rows():
    Q, K, _ = _head()
    pr = P.probe_rows(Q, K, 512)
    assert np.allclose(pr.vert.sum(axis=1), 16.0, atol=1e-4)
    assert np.allclose(pr.slash.sum(axis=1), 16.0, atol=1e-4)
    assert np.allclose(pr.P.sum(axis=1), 1.0, atol=1e-12)


def test_against_full_attention_matrix():
    Q, K, V = _head(seed=4, n=384)
    for q1 in (384, 256):                      # full sequence and a shorter segment end
        pr = P.probe_rows(Q, K, q1)
        Am = A.attention_matrix(Q, K)
        rows = np.arange(q1 - 64, q1)
        for g in range(4):
            rg = rows[16 * g:16 * g + 16]
            assert np.allclose(pr.vert[g], Am[rg][:, :q1].sum(axis=0), atol=1e-6)
            want = np.zeros(q1)
            for i in rg:
                for o in range(i + 1):
                    want[o] += Am[i, i - o]
            assert np.allclose(pr.slash[g], want, atol=1e-6)
        _, lse = A.dense_attention(Q, K, V, rows)
        assert np.allclose(pr.lse, lse, atol=1e-6)


def test_slash_offset_zero_is_the_diagonal_mass():
    Q, K, _ = _head(seed=5, n=256)
    pr = P.probe_rows(Q, K, 256)
    Am = A.attention_matrix(Q, K)
    assert abs(pr.slash[:, 0].sum() - np.diag(Am)[-64:].sum()) < 1e-5
    # a key at distance o from the last row is reached by exactly min(64, ...) rows
    assert pr.slash[:, 255].sum() == np.float32(Am[255, 0])


def test_pooling_and_block_scores_brute_force():
    Q, K, V = _head(seed=6, n=256)
    qp, kp = P.pool_mean(Q), P.pool_mean(K)
    for b in range(4):
        assert np.allclose(qp[b], sum(Q[64 * b + t] for t in range(64)) / 64)
        assert np.allclose(kp[b], sum(K[64 * b + t] for t in range(64)) / 64)
    s = P.block_scores(Q, K, 128, 256)
    assert s.shape == (2, 4)
    assert abs(s[0, 1] - float(qp[2] @ kp[1]) / np.sqrt(128)) < 1e-6
    assert s[0, 3] == -np.inf and s[1, 3] > -np.inf
    vn, vmax = P.value_norms(V, 256)
    assert abs(vn[7] - np.sqrt(sum(x * x for x in V[7]))) < 1e-5 and vmax == vn.max()


def test_descriptors_on_known_distributions():
    # K = 0 makes every probe row uniform over its causal keys
    Q, K, _ = _head(seed=7, n=2048)
    pr = P.probe_rows(Q, np.zeros_like(K), 2048)
    rows = np.arange(2048 - 64, 2048)
    assert abs(pr.entropy - np.log(rows + 1).mean()) < 1e-9
    assert abs(pr.local_conc - (1024 / (rows + 1)).mean()) < 1e-9


# ------------------------------------------------------------------ Eq. 3 in its general form (mixture rows, pooled keys)
def test_mixture_rows_are_distinct_ordered_and_inside_the_segment():
    for q0, q1 in ((0, 4096), (1024, 3072), (320, 384), (0, 64)):
        rows = P.mixture_rows(q0, q1)
        assert len(rows) == 64 and len(set(rows.tolist())) == 64
        assert rows.min() >= q0 and rows.max() == q1 - 1
        assert np.array_equal(rows[:32], np.arange(q1 - 32, q1))          # recent
        assert np.array_equal(rows[48:], np.arange(q0, q0 + 16))          # boundary-adjacent
        assert np.all(np.diff(rows[32:48]) > 0) and rows[32] >= q0 + 16 and rows[47] < q1 - 32
    # strata midpoints: the uniform rows of a long segment are evenly spaced
    rows = P.mixture_rows(0, 4096 + 48)
    assert set(np.diff(rows[32:48]).tolist()) == {256}


def test_pooled_probe_with_width_one_is_the_exact_probe():
    Q, K, _ = _head(seed=9, n=384)
    for q1 in (384, 256):
        pp = P.pooled_probe(Q, K, np.arange(q1 - 64, q1), 1, q1, [0, 16, 32, 48, 64])
        pr = P.probe_rows(Q, K, q1)
        assert np.allclose(pp.A, pr.P, atol=1e-12)
        assert np.allclose(pp.colmass, pr.vert, atol=1e-6) and np.allclose(pp.diagmass, pr.slash, atol=1e-6)
        assert np.allclose(pp.lse, pr.lse, atol=1e-5)
        assert abs(pp.local_conc - pr.local_conc) < 1e-9


def test_pooled_logit_is_the_mean_of_the_visible_per_key_logits():
    Q, K, _ = _head(seed=10, n=256)
    rows = np.array([255, 130, 77, 8, 3])
    g = 8
    S = P.pooled_logits(Q, K, rows, g, 256)
    for t, i in enumerate(rows):
        per_key = (K[:i + 1] @ Q[i]) / np.sqrt(128.0)                     # brute force, key by key
        for kb in range(256 // g):
            vis = per_key[kb * g:min(kb * g + g, i + 1)]
            if len(vis) == 0:
                assert S[t, kb] == -np.inf
            else:
                assert abs(S[t, kb] - vis.mean()) < 1e-10


def test_pooled_probe_on_identical_keys_is_uniform():
    rng = np.random.default_rng(5)
    n, g = 512, 16
    Q = rng.standard_normal((n, 128))
    K = np.tile(rng.standard_normal((1, 128)), (n, 1))
    rows = P.mixture_rows(0, n)
    pp = P.pooled_probe(Q, K, rows, g, n, [0, 32, 48, 64])
    for t, i in enumerate(rows):
        vis = i // g + 1
        assert np.allclose(pp.A[t, :vis], 1.0 / vis, atol=1e-12) and np.all(pp.A[t, vis:] == 0)
    # normalised entropy of a uniform row is 1 when it sees at least two blocks, 0 when it sees one
    want = np.mean([1.0 if i // g + 1 >= 2 else 0.0 for i in rows])
    assert abs(pp.entropy - want) < 1e-12
    # local-band mass of a uniform row = share of its visible blocks whose first key lies within 1024 of the row
    local = [sum(1 for kb in range(i // g + 1) if i - kb * g < 1024) / (i // g + 1) for i in rows]
    assert abs(pp.local_conc - np.mean(local)) < 1e-12


def test_pooled_probe_invariants():
    Q, K, _ = _head(seed=11, n=1024)
    rows = P.mixture_rows(0, 1024)
    for g in (8, 64):
        pp = P.pooled_probe(Q, K, rows, g, 1024, [0, 32, 48, 64])
        assert np.allclose(pp.A.sum(axis=1), 1.0, atol=1e-12)
        assert np.allclose(pp.colmass.sum(axis=1), [32, 16, 16]) and np.allclose(pp.diagmass.sum(axis=1), [32, 16, 16])
        assert 0.0 <= pp.entropy <= 1.0 and 0.0 <= pp.local_conc <= 1.0 + 1e-12 and 0.0 <= pp.agreement <= 1.0
        for t, i in enumerate(rows[:4]):
            assert abs(P.row_signature(pp.A[t], int(i), g).sum() - 1.0) < 1e-12
    # two subsets made of the same rows agree completely
    same = np.concatenate([rows[:16], rows[:16]])
    pp = P.pooled_probe(Q, K, same, 8, 1024, [0, 16, 32])
    assert abs(pp.agreement - 1.0) < 1e-12
    # a local head (recent and uniform rows both attend to their own neighbourhood) agrees more than a head whose
    # recent rows look at the neighbourhood and whose earlier rows look at key block 0
    n, g = 1024, 8
    Kl = np.zeros((n, 128)); Ql = np.zeros((n, 128))
    for j in range(n):
        Kl[j, j % 128] = 30.0
        Ql[j, j % 128] = 30.0                                             # row i likes keys j = i mod 128: a slash pattern
    a_local = P.pooled_probe(Ql, Kl, rows, g, n, [0, 32, 48, 64]).agreement
    Qm = Ql.copy()
    Qm[:n - 32] = 0.0
    Qm[:n - 32, 0] = 30.0                                                 # earlier rows like dim 0 = keys 0, 128, ...
    Km = Kl.copy()
    Km[1:, 0] = 0.0                                                       # ... of which only key 0 is left
    a_mixed = P.pooled_probe(Qm, Km, rows, g, n, [0, 32, 48, 64]).agreement
    assert a_local > a_mixed + 0.2


def test_probe_on_runs_of_the_query_mixture_against_the_full_attention_matrix():
    """The probe on four arbitrary 16-row runs (the query mixture at key resolution): column and diagonal masses by
    brute force from the full matrix A; with the runs of the last 64 rows it is the last-64-query probe."""
    Q, K, V = _head(seed=8, n=448)
    Am = A.attention_matrix(Q, K)
    for q0, q1 in ((0, 448), (128, 320)):
        starts = P.mixture_runs(q0, q1)
        assert starts[0] == q0 and starts[3] == q1 - 16 and np.all(np.diff(starts) >= 16) and np.all(starts % 16 == 0)
        pr = P.probe_rows(Q, K, q1, starts)
        for g, s0 in enumerate(starts):
            rg = np.arange(s0, s0 + 16)
            assert np.allclose(pr.vert[g], Am[rg][:, :q1].sum(axis=0), atol=1e-6)
            want = np.zeros(q1)
            for i in rg:
                for o in range(i + 1):
                    want[o] += Am[i, i - o]
            assert np.allclose(pr.slash[g], want, atol=1e-6)
            assert np.all(pr.slash[g, s0 + 16:] == 0)                # no row of the run reaches that far back
        _, lse = A.dense_attention(Q, K, V, np.concatenate([np.arange(s0, s0 + 16) for s0 in starts]))
        assert np.allclose(pr.lse, lse, atol=1e-6)
    a, b = P.probe_rows(Q, K, 320), P.probe_rows(Q, K, 320, [256, 272, 288, 304])
    assert np.array_equal(a.vert, b.vert) and np.array_equal(a.slash, b.slash) and np.array_equal(a.lse, b.lse)
    # thirds of the segment, in units of 16 rows
    assert P.mixture_runs(0, 64).tolist() == [0, 16, 32, 48]
    assert P.mixture_runs(64, 64 + 960).tolist() == [64, 64 + 320, 64 + 640, 64 + 944]


def test_agreement_descriptor_in_a_closed_form_case():
    """Recent rows that put all their mass on key block 0 (a sink 60 logits above everything else) against uniform-group
    rows whose queries are zero (uniform over the visible blocks): the recent signature is the unit vector of the
    [block 0] bin, a uniform row with v > 17 visible blocks has 1/v in that bin, so the total-variation distance is
    1 - mean(1/v) and agreement = mean(1/v).  Entropy: 0 for the recent rows, 1 for the uniform ones."""
    n, d, g = 64 * 40, 128, 64
    K = np.zeros((n, d)); Q = np.zeros((n, d))
    u = np.zeros(d); u[3] = 1.0
    K[:64] = u                                              # block 0: the sink direction, every other key is zero
    rows = np.array([n - 4, n - 3, n - 2, n - 1, 64 * 20 + 5, 64 * 25 + 63, 64 * 30])
    Q[rows[:4]] = 60.0 * np.sqrt(d) * u                     # logit 60 on block 0, 0 elsewhere
    pp = P.pooled_probe(Q, K, rows, g, n, [0, 4, 7])
    vis = np.array([21, 26, 31])
    assert abs(pp.agreement - np.mean(1.0 / vis)) < 1e-12
    assert abs(pp.entropy - 3.0 / 7.0) < 1e-12
    # identical groups agree completely; disjoint supports not at all
    same = P.pooled_probe(Q, K, rows[[0, 1, 2, 3]], g, n, [0, 2, 4])
    assert abs(same.agreement - 1.0) < 1e-12
    Q2 = Q.copy(); K2 = K.copy()
    K2[64 * 39:] = u; K2[:64] = 0.0                         # second pair of rows: all mass on their own block instead
    sig_a = P.row_signature(np.eye(40)[0], n - 1, g)        # everything on block 0 -> bin 0
    sig_b = P.row_signature(np.eye(40)[39], n - 1, g)       # everything on the row's own block -> offset 0 -> bin 1
    assert sig_a.tolist() == [1.0] + [0.0] * 17 and sig_b.tolist() == [0.0, 1.0] + [0.0] * 16
    assert P.row_signature(np.eye(40)[10], n - 1, g)[17] == 1.0          # far from both ends -> the [rest] bin
    assert P.row_signature(np.eye(40)[24], n - 1, g)[1 + 15] == 1.0      # relative offset 15 is still local
