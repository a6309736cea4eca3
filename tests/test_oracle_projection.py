"""Pins for the oracle's QKV projection with rotary embedding (the step in front of the probe). CPU only."""
import numpy as np
import torch

from oracle import projection as PJ


def _case(n=96, dm=64, Hq=4, Hkv=2, d=16, seed=0):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, dm))
    W = rng.standard_normal(((Hq + 2 * Hkv) * d, dm)) / np.sqrt(dm)
    cos, sin = PJ.rope_tables(n, d, base=10000.0)
    return X, W, cos, sin, Hq, Hkv, d


def test_projection_matches_torch_linear_and_rotate_half():
    """torch: F.linear, then x cos + rotate_half(x) sin with the tables repeated over both halves -- the formula
    Llama-family code uses, written with library ops (a transposed weight, a swapped sign or a wrong pairing fails)."""
    X, W, cos, sin, Hq, Hkv, d = _case()
    Q, K, V = PJ.qkv_project(X, W, cos, sin, Hq, Hkv, d)
    Y = torch.nn.functional.linear(torch.from_numpy(X), torch.from_numpy(W))          # [n, (Hq + 2 Hkv) d]
    Y = Y.view(X.shape[0], Hq + 2 * Hkv, d).transpose(0, 1)                            # [heads, n, d]
    c = torch.from_numpy(np.concatenate([cos, cos], axis=1)).double()
    s = torch.from_numpy(np.concatenate([sin, sin], axis=1)).double()
    rot = lambda x: torch.cat([-x[..., d // 2:], x[..., :d // 2]], dim=-1)
    R = Y * c + rot(Y) * s
    assert np.allclose(Q, R[:Hq].numpy(), atol=1e-12)
    assert np.allclose(K, R[Hq:Hq + Hkv].numpy(), atol=1e-12)
    assert np.allclose(V, Y[Hq + Hkv:].numpy(), atol=1e-12)                            # values are not rotated


def test_rope_special_cases():
    X, W, cos, sin, Hq, Hkv, d = _case(n=40)
    x = np.random.default_rng(1).standard_normal((40, d))
    # token 0 is not rotated; cos = 1, sin = 0 is the identity
    assert np.allclose(PJ.rope(x, cos, sin)[0], x[0])
    assert np.array_equal(PJ.rope(x, np.ones_like(cos), np.zeros_like(sin)), x)
    # a rotation: every (i, i + d/2) pair keeps its norm
    r = PJ.rope(x, cos, sin)
    h = d // 2
    assert np.allclose(r[:, :h] ** 2 + r[:, h:] ** 2, x[:, :h] ** 2 + x[:, h:] ** 2)
    # a quarter turn on one pair: (a, b) -> (-b, a)
    c1, s1 = np.zeros((1, h), np.float32), np.ones((1, h), np.float32)
    v = np.arange(d, dtype=np.float64)[None, :]
    assert np.allclose(PJ.rope(v, c1, s1), np.concatenate([-v[:, h:], v[:, :h]], axis=1))


def test_rotated_dot_products_depend_on_the_distance_only():
    """The property rotary embeddings exist for: <rope(q, i), rope(k, j)> is a function of i - j."""
    d, n = 16, 64
    cos, sin = PJ.rope_tables(n, d, base=100.0)
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    Qr = PJ.rope(np.tile(q, (n, 1)), cos, sin)
    Kr = PJ.rope(np.tile(k, (n, 1)), cos, sin)
    S = Qr @ Kr.T
    for delta in (0, 1, 7, 20):
        diag = np.array([S[i, i - delta] for i in range(delta, n)])
        assert np.allclose(diag, diag[0], atol=1e-5)          # tables are float32


def test_side_outputs_by_brute_force():
    rng = np.random.default_rng(3)
    A = rng.standard_normal((192, 8))
    bm = PJ.block_means(A)
    bn = PJ.block_max_sq_norm(A)
    for b in range(3):
        rows = A[64 * b:64 * b + 64]
        assert np.allclose(bm[b], sum(rows) / 64.0)
        assert np.isclose(bn[b], max(float(np.dot(r, r)) for r in rows))
