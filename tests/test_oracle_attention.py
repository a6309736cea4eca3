"""Pins for the oracle's dense (Eq. 1) and masked (Section 2.1) attention. CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as A
from synth import bf16_bits_to_f64, make_layer, tiny_spec


def _head(seed=3, n=256, d=128):
    L = make_layer(tiny_spec(seed, n, 1, 1, d))
    return (bf16_bits_to_f64(L["Q"][0]), bf16_bits_to_f64(L["K"][0]), bf16_bits_to_f64(L["V"][0]))


def test_row0_is_v0():
    Q, K, V = _head()
    O, lse = A.dense_attention(Q, K, V)
    assert np.array_equal(O[0], V[0].astype(np.float32))
    assert abs(lse[0] - (Q[0] @ K[0]) / math.sqrt(128)) < 1e-5


def test_zero_keys_give_running_mean():
    Q, K, V = _head(n=128)
    O, lse = A.dense_attention(Q, np.zeros_like(K), V)
    want = np.cumsum(V, axis=0) / np.arange(1, 129)[:, None]
    assert np.allclose(O, want, atol=1e-6)
    assert np.allclose(lse, np.log(np.arange(1, 129)), atol=1e-6)


def test_rows_of_A_sum_to_one_and_are_causal():
    Q, K, _ = _head(n=192)
    Am = A.attention_matrix(Q, K)
    assert np.allclose(Am.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(np.triu(Am, 1) == 0)


def test_matches_torch_sdpa():
    Q, K, V = _head(seed=5, n=512)
    O, _ = A.dense_attention(Q, K, V)
    q, k, v = (torch.from_numpy(x.astype(np.float32))[None, None] for x in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)[0, 0].numpy()
    assert np.abs(O - ref).max() < 1e-5


def test_pure_python_brute_force():
    rng = np.random.default_rng(0)
    n, d = 9, 4
    Q, K, V = rng.standard_normal((3, n, d))
    O, lse = A.dense_attention(Q, K, V)
    for i in range(n):
        ws = [math.exp(sum(Q[i][t] * K[j][t] for t in range(d)) / math.sqrt(d)) for j in range(i + 1)]
        Z = sum(ws)
        for t in range(d):
            assert abs(O[i][t] - sum(ws[j] * V[j][t] for j in range(i + 1)) / Z) < 1e-6
        assert abs(lse[i] - math.log(Z)) < 1e-6


def test_all_ones_mask_reproduces_dense_bitwise():
    Q, K, V = _head(seed=7, n=320)
    O, lse = A.dense_attention(Q, K, V)
    Om, lsem, onorm = A.masked_attention(Q, K, V, lambda r, nk: np.ones((len(r), nk), bool))
    assert np.array_equal(O, Om) and np.array_equal(lse, lsem)
    assert np.allclose(onorm, np.linalg.norm(O.astype(np.float64), axis=1), rtol=1e-6)


def test_lse_merge_of_a_key_split_reproduces_the_unsplit_row():
    Q, K, V = _head(seed=9, n=256)
    rows = np.arange(64, 256)
    O, lse = A.dense_attention(Q, K, V, rows)
    # the first part keeps key 0 so that no row is empty
    part1 = lambda r, nk: np.broadcast_to((np.arange(nk) % 3 == 0)[None, :], (len(r), nk)).copy()
    part2 = lambda r, nk: ~part1(r, nk)
    O1, l1, _ = A.masked_attention(Q, K, V, part1, rows)
    O2, l2, _ = A.masked_attention(Q, K, V, part2, rows)
    l1, l2 = l1.astype(np.float64), l2.astype(np.float64)
    lm = np.logaddexp(l1, l2)
    Om = np.exp(l1 - lm)[:, None] * O1 + np.exp(l2 - lm)[:, None] * O2
    assert np.allclose(lm, lse, atol=1e-5)
    assert np.allclose(Om, O, atol=1e-5)


def test_explicit_bitset_brute_force():
    rng = np.random.default_rng(1)
    n, d = 48, 8
    Q, K, V = rng.standard_normal((3, n, d))
    M = rng.random((n, n)) < 0.3
    M[np.arange(n), np.arange(n)] = True
    O, lse, onorm = A.masked_attention(Q, K, V, lambda r, nk: M[r][:, :nk])
    for i in range(n):
        js = [j for j in range(i + 1) if M[i, j]]
        ws = np.array([math.exp(float(Q[i] @ K[j]) / math.sqrt(d)) for j in js])
        o = (ws[:, None] * V[js]).sum(0) / ws.sum()
        assert np.allclose(O[i], o, atol=1e-6)
        assert abs(lse[i] - math.log(ws.sum())) < 1e-6
        assert abs(onorm[i] - np.linalg.norm(o)) < 1e-6


def test_transposed_operands_would_fail():
    """Swapping Q and K changes the result on asymmetric inputs: guards against a transposed product."""
    Q, K, V = _head(seed=11, n=128)
    O, _ = A.dense_attention(Q, K, V)
    Ot, _ = A.dense_attention(K, Q, V)
    assert np.abs(O - Ot).max() > 1e-2


def test_relative_error_eq9():
    O = np.array([[3.0, 4.0]])
    assert abs(A.relative_error(O, O) - 0.0) < 1e-15
    assert abs(A.relative_error(O, np.zeros_like(O)) - 1.0) < 1e-12
