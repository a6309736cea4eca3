"""GPU test of rs_dense_prefill_attn_noalloc, the entry point for callers that cannot allocate device memory
(plugins that only get their tensors, allocator callbacks, serving loops where cudaMalloc is off limits).

It must give what rs_dense_prefill_attn gives, on two calls in a row (the built-in scratch is shared and keeps the
previous call's contents), and must refuse problems larger than its fixed scratch.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import ATOL_MAX, ATOL_MEAN, dev_bf16
from synth import make_layer, tiny_spec

pytestmark = pytest.mark.gpu


def _reference(p, Q, K, V):
    O = torch.zeros((p.n_q_heads, p.n_keys, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((p.n_q_heads, p.n_keys), dtype=torch.float32, device="cuda")
    onorm = torch.zeros_like(lse)
    st = rs.new_status()
    rs.rs_dense_prefill_attn(p, Q, K, V, O, lse, onorm, None, rs.new_workspace(p, None), st)
    rs.check_status(st, "dense")
    return O.cpu().numpy(), lse.cpu().numpy(), onorm.cpu().numpy()


def _noalloc(p, Q, K, V):
    O = torch.zeros((p.n_q_heads, p.n_keys, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((p.n_q_heads, p.n_keys), dtype=torch.float32, device="cuda")
    onorm = torch.zeros_like(lse)
    st = rs.new_status()
    rs.rs_dense_prefill_attn_noalloc(p, Q, K, V, O, lse, onorm, st)
    rs.check_status(st, "dense without allocation")
    return O.cpu().numpy(), lse.cpu().numpy(), onorm.cpu().numpy()


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    cases = [(1088, 4, 2, [0, 1088]), (704, 2, 1, [0, 192, 704])]      # the second call reuses the scratch of the first
    for n, Hq, Hkv, bounds in cases:
        L = make_layer(tiny_spec(90 + n, n, Hq, Hkv))
        p = rs.Problem(Hq, Hkv, n, bounds)
        Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
        want = _reference(p, Q, K, V)
        for call in range(2):
            got = _noalloc(p, Q, K, V)
            err = np.abs(got[0] - want[0])
            assert err.max() <= ATOL_MAX and err.mean() <= ATOL_MEAN, (n, call, err.max())
            assert np.abs(got[1] - want[1]).max() < 2e-3
            assert np.all(np.abs(got[2] - want[2]) <= 1e-2 * np.abs(want[2]) + 1e-3)


def test_sizes_beyond_the_built_in_scratch_are_refused():
    p = rs.Problem(32, 8, 131072)                     # 32 heads x 1024 tiles = 32768 > 16384
    x = torch.zeros(8, device="cuda")
    with pytest.raises(rs.RouteSparseError, match="no-allocation"):
        rs.rs_dense_prefill_attn_noalloc(p, x, x, x, x, x, None, None)
