"""GPU test of rs_dense_prefill_attn_noalloc, the entry point for callers that cannot allocate device memory
(plugins that only get their tensors, allocator callbacks, serving loops where cudaMalloc is off limits).

It must give what rs_dense_prefill_attn gives, on two calls in a row (the built-in scratch is shared and keeps the
previous call's contents), and must refuse problems larger than its fixed scratch.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import assert_attention_close, dev_bf16, f64_heads
from oracle import attention as A
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu


def _run(entry, p, Q, K, V):
    O = torch.zeros((p.n_q_heads, p.n_keys, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((p.n_q_heads, p.n_keys), dtype=torch.float32, device="cuda")
    onorm = torch.zeros_like(lse)
    st = rs.new_status()
    if entry == "workspace":
        rs.rs_dense_prefill_attn(p, Q, K, V, O, lse, onorm, None, rs.new_workspace(p, None), st)
    else:
        rs.rs_dense_prefill_attn_noalloc(p, Q, K, V, O, lse, onorm, st)
    rs.check_status(st, entry)
    return O, lse, onorm


def test_two_calls_in_a_row_match_the_oracle_and_the_workspace_entry_point():
    """Two different problems, each called twice in a row: the second call of a problem and the first call of the next
    one find the previous call's work list in the built-in scratch.  Each result is compared with the oracle's dense
    attention (Eq. 1) at the tolerance of the other attention tests, and must equal rs_dense_prefill_attn's result bit
    for bit: both run the same kernels on the same work list, only the scratch lives elsewhere."""
    cases = [(1088, 4, 2, [0, 1088]), (704, 2, 1, [0, 192, 704])]
    for n, Hq, Hkv, bounds in cases:
        L = make_layer(tiny_spec(90 + n, n, Hq, Hkv))
        p = rs.Problem(Hq, Hkv, n, bounds)
        Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
        want = _run("workspace", p, Q, K, V)
        Qs, Ks, Vs = f64_heads(L)
        oracle = [A.dense_attention(Qs[h], Ks[h // (Hq // Hkv)], Vs[h // (Hq // Hkv)]) for h in range(Hq)]
        for call in range(2):
            got = _run("no allocation", p, Q, K, V)
            for h in range(Hq):
                Oo, lo = oracle[h]
                assert_attention_close(got[0][h].cpu().numpy(), Oo, f"n={n} call {call} head {h}")
                assert np.abs(got[1][h].cpu().numpy() - lo).max() < 2e-3
                ref_norm = np.linalg.norm(Oo.astype(np.float64), axis=1)
                assert np.all(np.abs(got[2][h].cpu().numpy() - ref_norm) < 1e-2 * ref_norm + 1e-3)
            for a, b in zip(got, want):
                assert torch.equal(a, b), (n, call)


def test_the_limit_itself_is_accepted_and_one_head_more_is_refused():
    """heads x 128-row tiles == 16384 uses the last entries of the built-in scratch; one head more does not fit."""
    n = 512                                            # 4 tiles per head
    Hq, Hkv = 4096, 1024                               # 4096 x 4 = 16384 tiles
    gen = torch.Generator(device="cuda").manual_seed(5)
    mk = lambda H: torch.randn((H, n, 128), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    Q, K, V = mk(Hq), mk(Hkv), mk(Hkv)
    p = rs.Problem(Hq, Hkv, n)
    got = _run("no allocation", p, Q, K, V)
    want = _run("workspace", p, Q, K, V)
    for a, b in zip(got, want):
        assert torch.equal(a, b)
    # the last heads (whose tiles sit at the end of the work list) against the oracle
    tof = lambda t: t.float().cpu().numpy().astype(np.float64)
    for h in (0, Hq - 1):
        Oo, lo = A.dense_attention(tof(Q[h]), tof(K[h // 4]), tof(V[h // 4]))
        assert_attention_close(got[0][h].cpu().numpy(), Oo, f"head {h}")
        assert np.abs(got[1][h].cpu().numpy() - lo).max() < 2e-3
    p_over = rs.Problem(Hq + 4, Hkv + 1, n)            # 16400 tiles
    x = torch.zeros(8, device="cuda")
    with pytest.raises(rs.RouteSparseError, match="no-allocation"):
        rs.rs_dense_prefill_attn_noalloc(p_over, x, x, x, x, x, None, None)


def test_sizes_beyond_the_built_in_scratch_are_refused():
    p = rs.Problem(32, 8, 131072)                     # 32 heads x 1024 tiles = 32768 > 16384
    x = torch.zeros(8, device="cuda")
    with pytest.raises(rs.RouteSparseError, match="no-allocation"):
        rs.rs_dense_prefill_attn_noalloc(p, x, x, x, x, x, None, None)
