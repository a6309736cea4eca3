"""GPU parity: rs_dense_prefill_attn / rs_sparse_prefill_attn against the oracle under the same mask.

Tolerance: bf16 inputs, fp32 accumulation, bf16 P: max-abs 2e-2 and mean-abs 5e-3 on the attention output;
log-sum-exp within 2e-3 absolute (fp32 exp2/log2 of sums of up to n terms).
"""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import (assert_attention_close, c_library, dev_bf16, f64_heads, oracle_index_sets,
                         oracle_probe_all, upload_materialised)
from oracle import attention as A
from oracle import patterns as PT
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu
C = PT.Candidate


def _run_dense(L, p, out_dtype):
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    ws = rs.new_workspace(p, None)
    O = torch.zeros((p.n_q_heads, p.n_keys, 128), dtype=out_dtype, device="cuda")
    lse = torch.zeros((p.n_q_heads, p.n_keys), dtype=torch.float32, device="cuda")
    onorm = torch.zeros_like(lse)
    st = rs.new_status()
    cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
    rs.rs_dense_prefill_attn(p, Q, K, V, O, lse, onorm, cnt, ws, st)
    rs.check_status(st, "dense")
    return O.float().cpu().numpy(), lse.cpu().numpy(), onorm.cpu().numpy(), cnt.cpu().numpy()


@pytest.mark.parametrize("n,Hq,Hkv", [(64, 1, 1), (192, 2, 1), (1088, 4, 2)])
def test_dense_matches_oracle(n, Hq, Hkv):
    L = make_layer(tiny_spec(11 + n, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n)
    O, lse, onorm, cnt = _run_dense(L, p, torch.float32)
    Qs, Ks, Vs = f64_heads(L)
    for h in range(Hq):
        g = h // (Hq // Hkv)
        Oo, lo = A.dense_attention(Qs[h], Ks[g], Vs[g])
        assert_attention_close(O[h], Oo, f"dense h={h}")
        assert np.abs(lse[h] - lo).max() < 2e-3
        ref_norm = np.linalg.norm(Oo.astype(np.float64), axis=1)
        assert np.all(np.abs(onorm[h] - ref_norm) < 1e-2 * ref_norm + 1e-3)
    nb = n // 64
    tiles = (n + 127) // 128
    assert cnt[1] == Hq * tiles
    assert cnt[0] == Hq * sum(min(nb, 2 * t + 2) for t in range(tiles))


def test_dense_bf16_output_and_segments():
    n, Hq, Hkv = 576, 2, 2
    L = make_layer(tiny_spec(5, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, [0, 192, 576])       # a segment boundary that is not a multiple of 128
    O32, lse, _, _ = _run_dense(L, p, torch.float32)
    Qs, Ks, Vs = f64_heads(L)
    for h in range(Hq):
        Oo, lo = A.dense_attention(Qs[h], Ks[h], Vs[h])
        assert_attention_close(O32[h], Oo, f"dense, segments, h={h}")
        assert np.abs(lse[h] - lo).max() < 2e-3
    # the bf16 output is the same result rounded once (round to nearest even): bit-identical to rounding the fp32 output
    O16, lse16, _, _ = _run_dense(L, p, torch.bfloat16)
    assert np.array_equal(O16, torch.from_numpy(O32).to(torch.bfloat16).float().numpy())
    assert np.array_equal(lse16, lse)


CANDS = [C(PT.DENSE), C(PT.A_SHAPE, 8, 96), C(PT.A_SHAPE, 70, 200), C(PT.VERTICAL_SLASH, 24, 40),
         C(PT.VERTICAL_SLASH, 100, 6), C(PT.BLOCK_SPARSE, 3), C(PT.BLOCK_SPARSE, 1), C(PT.A_SHAPE, 0, 1)]


@pytest.mark.parametrize("seg_bounds", [[0, 832], [0, 320, 832]])
def test_sparse_patterns_match_oracle_under_the_same_mask(seg_bounds):
    n, Hq, Hkv = 832, 8, 2
    L = make_layer(tiny_spec(17, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, seg_bounds)
    Qs, Ks, Vs = f64_heads(L)
    probes = oracle_probe_all(Qs, Ks, p)
    rng = np.random.default_rng(3)
    choice = [(item + 3 * (item // Hq)) % len(CANDS) for item in range(p.n_items)]
    sets = oracle_index_sets(p, CANDS, choice, probes)
    lib = c_library(CANDS)
    idx = upload_materialised(p, lib, sets)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    ws = rs.new_workspace(p, lib)
    O = torch.zeros((Hq, n, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((Hq, n), dtype=torch.float32, device="cuda")
    onorm = torch.zeros_like(lse)
    st = rs.new_status()
    ch = torch.tensor(choice, dtype=torch.int32, device="cuda")
    rs.rs_sparse_prefill_attn(p, Q, K, V, lib, idx, ch, O, lse, onorm, None, ws, st)
    rs.check_status(st, "sparse")
    O, lse, onorm = O.cpu().numpy(), lse.cpu().numpy(), onorm.cpu().numpy()
    for item, ix in enumerate(sets):
        h = item % Hq
        g = h // (Hq // Hkv)
        rows = np.arange(ix.q0, ix.q1)
        Oo, lo, no = A.masked_attention(Qs[h], Ks[g], Vs[g], lambda r, nk: PT.mask_rows(ix, r, nk), rows)
        assert_attention_close(O[h, rows], Oo, f"item {item} {ix.cand}")
        assert np.abs(lse[h, rows] - lo).max() < 2e-3, ix.cand
        assert np.all(np.abs(onorm[h, rows] - no) < 1e-2 * no + 1e-3)


def test_argument_checks():
    p = rs.Problem(2, 1, 100)
    with pytest.raises(rs.RouteSparseError):
        rs.rs_workspace_bytes(p, None)
    p = rs.Problem(2, 1, 128)
    x = torch.zeros(16, device="cuda")
    with pytest.raises(rs.RouteSparseError):      # workspace too small
        rs.rs_dense_prefill_attn(p, x, x, x, x, x, None, None, torch.zeros(256, dtype=torch.uint8, device="cuda")[:0]
                                 if False else torch.zeros(256, dtype=torch.uint8, device="cuda")[:128], None)


def test_single_block_and_maximum_length():
    """Degenerate sizes: one 64-row block under every pattern, and the largest supported length (262144 keys)."""
    L = make_layer(tiny_spec(3, 64, 1, 1))
    p = rs.Problem(1, 1, 64)
    Qs, Ks, Vs = f64_heads(L)
    cands = [C(PT.A_SHAPE, 4, 8), C(PT.VERTICAL_SLASH, 7, 5), C(PT.BLOCK_SPARSE, 1), C(PT.DENSE)]
    probes = oracle_probe_all(Qs, Ks, p)
    for c in range(len(cands)):
        sets = oracle_index_sets(p, cands, [c], probes)
        lib = c_library(cands)
        idx = upload_materialised(p, lib, sets)
        O = torch.zeros((1, 64, 128), dtype=torch.float32, device="cuda")
        lse = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
        st = rs.new_status()
        rs.rs_sparse_prefill_attn(p, dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"]), lib, idx,
                                  torch.tensor([c], dtype=torch.int32, device="cuda"), O, lse, None, None,
                                  rs.new_workspace(p, lib), st)
        rs.check_status(st, "single block")
        Oo, lo, _ = A.masked_attention(Qs[0], Ks[0], Vs[0], lambda r, nk: PT.mask_rows(sets[0], r, nk))
        assert_attention_close(O[0].cpu().numpy(), Oo, str(cands[c]))
    n = 262144
    L = make_layer(tiny_spec(4, n, 1, 1))
    p = rs.Problem(1, 1, n)
    cands = [C(PT.A_SHAPE, 128, 1024), C(PT.DENSE)]
    lib = c_library(cands)
    ix = PT.build_indices(cands[0], 0, n)
    idx = upload_materialised(p, lib, [ix])
    O = torch.zeros((1, n, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((1, n), dtype=torch.float32, device="cuda")
    st = rs.new_status()
    rs.rs_sparse_prefill_attn(p, dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"]), lib, idx,
                              torch.zeros(1, dtype=torch.int32, device="cuda"), O, lse, None, None, rs.new_workspace(p, lib), st)
    rs.check_status(st, "maximum length")
    Qs, Ks, Vs = f64_heads(L)
    for rows in (np.arange(0, 64), np.arange(100000, 100064), np.arange(n - 64, n)):
        Oo, lo, _ = A.masked_attention(Qs[0], Ks[0], Vs[0], lambda r, nk: PT.mask_rows(ix, r, nk), rows, chunk=64)
        assert_attention_close(O[0, rows].cpu().numpy(), Oo, f"rows {rows[0]}")
        assert np.abs(lse[0, rows].cpu().numpy() - lo).max() < 2e-3
    with pytest.raises(rs.RouteSparseError):
        rs.rs_workspace_bytes(rs.Problem(1, 1, 2 * n), None)


def test_many_vertical_columns_cover_both_mask_paths():
    """A vertical-slash head with more gathered columns than the per-tile keep masks cover (128 chunks = 8192 columns):
    the first chunks use the precomputed masks, the rest the per-element path; columns inside block diagonals are
    de-duplicated, columns after a row are invisible.  Checked on sampled rows against the oracle under the same mask."""
    n = 16384
    L = make_layer(tiny_spec(29, n, 1, 1))
    p = rs.Problem(1, 1, n)
    rng = np.random.default_rng(9)
    cand = C(PT.VERTICAL_SLASH, 9000, 3)
    V_cols = np.sort(rng.choice(n, 9000, replace=False)).astype(np.int32)
    S_offs = np.array([0, 70, 5000], dtype=np.int32)
    D = np.unique(np.concatenate([S_offs // 64, (S_offs + 63) // 64])).astype(np.int32)
    ix = PT.IndexSet(cand=cand, q0=0, q1=n, V=V_cols, S=S_offs, D=D)
    lib = c_library([cand, C(PT.DENSE)])
    idx = upload_materialised(p, lib, [ix])
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    O = torch.zeros((1, n, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((1, n), dtype=torch.float32, device="cuda")
    st = rs.new_status()
    rs.rs_sparse_prefill_attn(p, Q, K, V, lib, idx, torch.zeros(1, dtype=torch.int32, device="cuda"), O, lse, None, None,
                              rs.new_workspace(p, lib), st)
    rs.check_status(st, "many verticals")
    Qs, Ks, Vs = f64_heads(L)
    rows = np.concatenate([np.arange(0, 128), np.arange(5000, 5128), np.arange(9984, 10112), np.arange(n - 128, n)])
    Oo, lo, _ = A.masked_attention(Qs[0], Ks[0], Vs[0], lambda r, nk: PT.mask_rows(ix, r, nk), rows)
    assert_attention_close(O[0].cpu().numpy()[rows], Oo, "many verticals")
    assert np.abs(lse[0].cpu().numpy()[rows] - lo).max() < 2e-3
