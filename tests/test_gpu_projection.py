"""GPU parity: rs_qkv_rope_project (QKV projection + rotary embedding with the probe's side outputs fused into its
epilogue) against the oracle, and the probe fed by it against the probe that pools by itself.

Tolerances: Q, K, V are bf16 roundings of fp32-accumulated sums of 1e3..4e3 products of bf16 inputs: the oracle's
float64 value rounded to bf16 and the kernel's differ by at most one bf16 ulp where the two lie on either side of a
rounding boundary, i.e. |diff| <= 2^-8 |value| + tiny.  The side outputs are compared with the oracle's reduction OF
THE KERNEL'S OWN bf16 TENSORS (each stage fed what the previous GPU stage produced), at 1e-5 relative."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from oracle import projection as PJ
from oracle import probe as OP
from synth import bf16_bits_to_f64, f32_to_bf16_bits

pytestmark = pytest.mark.gpu


def _inputs(n, dm, Hq, Hkv, seed):
    rng = np.random.default_rng(seed)
    Xb = f32_to_bf16_bits(rng.standard_normal((n, dm)).astype(np.float32))
    Wb = f32_to_bf16_bits((rng.standard_normal(((Hq + 2 * Hkv) * 128, dm)) / np.sqrt(dm)).astype(np.float32))
    cos, sin = PJ.rope_tables(n, 128)
    return Xb, Wb, cos, sin


def _dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _run(Xb, Wb, cos, sin, Hq, Hkv, side=True):
    n = Xb.shape[0]
    bf = dict(dtype=torch.bfloat16, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    Q = torch.full((Hq, n, 128), 9.0, **bf); K = torch.full((Hkv, n, 128), 9.0, **bf); V = torch.full((Hkv, n, 128), 9.0, **bf)
    qpool = torch.full((Hq, n // 64, 128), 9.0, **f32) if side else None
    kpool = torch.full((Hkv, n // 64, 128), 9.0, **f32) if side else None
    vbmax = torch.full((Hkv, n // 64), 9.0, **f32) if side else None
    st = rs.new_status()
    rs.rs_qkv_rope_project(_dev_bf16(Xb), _dev_bf16(Wb), torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda(),
                           Hq, Hkv, Q, K, V, qpool, kpool, vbmax, st)
    rs.check_status(st, "projection")
    return Q, K, V, qpool, kpool, vbmax


@pytest.mark.parametrize("n,dm,Hq,Hkv", [(64, 64, 2, 2), (320, 192, 4, 2), (1088, 512, 8, 2)])
def test_projection_matches_oracle(n, dm, Hq, Hkv):
    Xb, Wb, cos, sin = _inputs(n, dm, Hq, Hkv, 100 + n)
    Q, K, V, qpool, kpool, vbmax = _run(Xb, Wb, cos, sin, Hq, Hkv)
    Qo, Ko, Vo = PJ.qkv_project(bf16_bits_to_f64(Xb), bf16_bits_to_f64(Wb), cos, sin, Hq, Hkv)
    for got, want in ((Q, Qo), (K, Ko), (V, Vo)):
        g = got.float().cpu().numpy().astype(np.float64)
        err = np.abs(g - want)
        assert np.all(err <= 2.0 ** -8 * np.abs(want) + 1e-6), float((err - 2.0 ** -8 * np.abs(want)).max())
        assert err.mean() <= 5e-3 and err.max() <= 2e-2 * max(1.0, np.abs(want).max())
    # side outputs: the oracle's reductions of the tensors the kernel wrote
    for h in range(Hq):
        assert np.allclose(qpool[h].cpu().numpy(), PJ.block_means(Q[h].float().cpu().numpy()), rtol=1e-5, atol=1e-6)
    for g in range(Hkv):
        assert np.allclose(kpool[g].cpu().numpy(), PJ.block_means(K[g].float().cpu().numpy()), rtol=1e-5, atol=1e-6)
        assert np.allclose(vbmax[g].cpu().numpy(), PJ.block_max_sq_norm(V[g].float().cpu().numpy()), rtol=1e-5)


def test_side_outputs_are_optional_and_the_run_is_deterministic():
    n, dm, Hq, Hkv = 320, 128, 4, 2
    Xb, Wb, cos, sin = _inputs(n, dm, Hq, Hkv, 7)
    a = _run(Xb, Wb, cos, sin, Hq, Hkv)
    b = _run(Xb, Wb, cos, sin, Hq, Hkv)
    c = _run(Xb, Wb, cos, sin, Hq, Hkv, side=False)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    for x, y in zip(a[:3], c[:3]):
        assert torch.equal(x, y)


def test_probe_fed_by_the_projection_equals_the_probe_that_pools_itself():
    """Q, K, V and the side outputs from the projection, then rs_probe without its own pooling / value-norm kernels
    (NULL outputs) and rs_value_norm_max: the masses are bit-identical to a probe call that pools by itself, the pooled
    keys and V_max agree with it and with the oracle to 1e-5."""
    n, dm, Hq, Hkv = 1088, 256, 4, 2
    Xb, Wb, cos, sin = _inputs(n, dm, Hq, Hkv, 11)
    Q, K, V, qpool, kpool, vbmax = _run(Xb, Wb, cos, sin, Hq, Hkv)
    p = rs.Problem(Hq, Hkv, n, [0, 320, 1088])
    S = p.n_segments
    f32 = dict(dtype=torch.float32, device="cuda")
    mk = lambda: (torch.zeros((S, Hq, 4, n), **f32), torch.zeros((S, Hq, 4, n), **f32), torch.zeros((Hq, S, 64), **f32))
    ws, st = rs.new_workspace(p, None), rs.new_status()
    v1, s1, l1 = mk()
    rs.rs_probe(p, Q, K, V, v1, s1, l1, None, None, None, None, ws, st)
    vmax1 = torch.zeros((S, Hkv), **f32)
    rs.rs_value_norm_max(p, vbmax, vmax1, st)
    v2, s2, l2 = mk()
    qp2 = torch.zeros((Hq, n // 64, 128), **f32); kp2 = torch.zeros((Hkv, n // 64, 128), **f32); vmax2 = torch.zeros((S, Hkv), **f32)
    rs.rs_probe(p, Q, K, V, v2, s2, l2, qp2, kp2, vmax2, None, ws, st)
    rs.check_status(st, "probe after projection")
    assert torch.equal(v1, v2) and torch.equal(s1, s2) and torch.equal(l1, l2)
    assert torch.allclose(kpool, kp2, rtol=1e-5, atol=1e-6) and torch.allclose(qpool, qp2, rtol=1e-5, atol=1e-6)
    assert torch.allclose(vmax1, vmax2, rtol=1e-5)
    Vf = V.float().cpu().numpy().astype(np.float64)
    for s in range(S):
        for g in range(Hkv):
            _, vm = OP.value_norms(Vf[g], p.seg_bounds[s + 1])
            assert abs(float(vmax1[s, g]) - vm) <= 1e-5 * vm


def test_argument_checks():
    x = torch.zeros(8, device="cuda")
    with pytest.raises(rs.RouteSparseError):
        rs.rs_qkv_rope_project(torch.zeros((100, 64), device="cuda", dtype=torch.bfloat16), x, x, x, 2, 2, x, x, x, None, None, None, None)
    with pytest.raises(rs.RouteSparseError):
        rs.rs_qkv_rope_project(torch.zeros((128, 64), device="cuda", dtype=torch.bfloat16), x, x, x, 3, 3, x, x, x, None, None, None, None)


def test_layer_pass_from_hidden_states_equals_the_pass_on_the_projected_tensors():
    """RoutedPrefillLayer.forward_from_hidden (projection with fused side outputs, probe without pooling) against the
    ordinary forward() on the Q, K, V the projection wrote: same routes, bit-identical output."""
    n, dm, Hq, Hkv = 1088, 256, 4, 2
    Xb, Wb, cos, sin = _inputs(n, dm, Hq, Hkv, 21)
    p = rs.Problem(Hq, Hkv, n)
    lib = [(rs.RS_A_SHAPE, 8, 128), (rs.RS_VERTICAL_SLASH, 32, 48), (rs.RS_BLOCK_SPARSE, 3, 0), (rs.RS_DENSE, 0, 0)]
    cfg = dict(budget_frac=0.4, cert_max=0.8)
    a = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(**cfg), out_dtype=torch.float32)
    Oa = a.forward_from_hidden(_dev_bf16(Xb), _dev_bf16(Wb), torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()).clone()
    rs.check_status(a.status, "from hidden")
    Q, K, V = a._qkv
    b = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(**cfg), out_dtype=torch.float32)
    b.one_call = False
    Ob = b.forward(Q, K, V)
    rs.check_status(b.status, "staged")
    assert torch.equal(a.choice, b.choice)
    assert torch.equal(Oa, Ob) and torch.equal(a.lse_sel, b.lse_sel)
    assert torch.equal(a.stats, b.stats)
