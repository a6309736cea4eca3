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
