"""GPU end-to-end: probe -> candidate evaluation -> routing -> materialisation -> attention -> certificate,
checked stage by stage against the oracle (each stage is fed what the previous GPU stage produced, so that a
1e-3 difference in probe scores cannot flip a later integer decision inside the comparison)."""
import numpy as np
import pytest
import torch

import paper_2608_29058_b200 as rs
from gpu_helpers import assert_attention_close, dev_bf16, f64_heads
from oracle import attention as A
from oracle import certificate as CT
from oracle import patterns as PT
from oracle import probe as OP
from oracle import routing as RT
from bench import download_sets
from synth import config1_spec, make_layer, tiny_spec

pytestmark = pytest.mark.gpu
C = PT.Candidate


def run_and_check(spec, bounds, cands, cfg, seed_name):
    L = make_layer(spec)
    Hq, Hkv, n = spec.n_q_heads, spec.n_kv_heads, spec.n
    p = rs.Problem(Hq, Hkv, n, bounds)
    layer = rs.RoutedPrefillLayer(p, [(c.pattern, c.b0, c.b1) for c in cands], cfg, out_dtype=torch.float32)
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    O = layer.forward(Q, K, V).cpu().numpy()
    rs.check_status(layer.status, seed_name)
    Qs, Ks, Vs = f64_heads(L)
    G = Hq // Hkv
    vert, slash = layer.vert.cpu().numpy(), layer.slash.cpu().numpy()
    stats = layer.stats.cpu().numpy()
    choice = layer.choice.cpu().numpy()
    # stage 2: candidate stats from the GPU's own probe scores (A-shape, vertical-slash, dense: bit-exact)
    cov = stats[:, :, :4].astype(np.uint64)
    pairs = stats[:, :, 4]
    for item in range(p.n_items):
        s, h = divmod(item, Hq)
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        for c, cand in enumerate(cands):
            if cand.pattern == PT.BLOCK_SPARSE:
                assert pairs[item, c] == sum((min(cand.b0, qb + 1) - 1) * 4096 + 2080 for qb in range(q0 // 64, q1 // 64))
                continue
            ix = PT.build_indices(cand, q0, q1, vert[s, h][:, :q1], slash[s, h][:, :q1], None)
            assert pairs[item, c] == PT.pairs(ix), (item, cand)
            if cand.pattern != PT.DENSE:
                assert cov[item, c].tolist() == PT.coverage_fx(ix, vert[s, h][:, :q1], slash[s, h][:, :q1]).tolist()
    # stage 3: routing from the GPU's stats
    vmax = layer.vmax.cpu().numpy()
    vmax_item = np.array([vmax[it // Hq, (it % Hq) // G] for it in range(p.n_items)], np.float32)
    want, wrep = RT.route(cands, cov, 512 * pairs, vmax_item, RT.RouteParams(
        budget=int(cfg.budget_frac * rs.dense_flops(p.seg_bounds, Hq)), t_probe=rs.probe_flops(p.seg_bounds, Hq),
        alpha=cfg.alpha, delta_q=cfg.delta_q, cert_max=cfg.cert_max, cert_mode=cfg.cert_mode,
        expand_first=cfg.expand_first))
    assert np.array_equal(choice, want)
    rep = layer.route_report()
    assert rep["total_cost"] == wrep.total_cost and rep["feasible"] == wrep.feasible and rep["n_fallback"] == wrep.n_fallback
    # stage 4: attention under the materialised index sets; stage 5: certificate against the true error
    sets = download_sets(layer, cands, choice)
    lse_sel, onorm = layer.lse_sel.cpu().numpy(), layer.onorm.cpu().numpy()
    m_head, cert_head = layer.m_head.cpu().numpy(), layer.cert_head.cpu().numpy()
    m_rows = layer.m_row.cpu().numpy()
    for item, ix in enumerate(sets):
        s, h = divmod(item, Hq)
        g = h // G
        rows = np.arange(ix.q0, ix.q1)
        if ix.cand.pattern == PT.VERTICAL_SLASH:      # lists equal the oracle's selection on the same scores
            ref = PT.build_indices(ix.cand, ix.q0, ix.q1, vert[s, h][:, :ix.q1], slash[s, h][:, :ix.q1], None)
            assert np.array_equal(ix.V, ref.V) and np.array_equal(ix.S, ref.S) and np.array_equal(ix.D, ref.D)
        Om, lo, no = A.masked_attention(Qs[h], Ks[g], Vs[g], lambda r, nk: PT.mask_rows(ix, r, nk), rows)
        assert_attention_close(O[h, rows], Om, f"item {item} {ix.cand}")
        assert np.abs(lse_sel[h, rows] - lo).max() < 2e-3
        Od, ld = A.dense_attention(Qs[h], Ks[g], Vs[g], rows)
        _, vm = OP.value_norms(Vs[g], n)
        m, cert, tight, _, _, _ = CT.certificate(lse_sel[h, rows], ld, vm, onorm[h, rows])
        # Eq. 5 on every row: the certificate built from the kernel's log-sum-exp bounds the exact error of the mask
        # (1e-2 absorbs the fp32 rounding of lse_sel, which enters as 2 * V_max * |d lse|)
        err = np.linalg.norm(Od.astype(np.float64) - Om.astype(np.float64), axis=1)
        assert np.all(cert + 1e-2 >= err), (item, ix.cand)
        # online certificate on the probe rows: kernel-side mass equals builder-side coverage
        if ix.cand.pattern != PT.DENSE:
            m_hat, _ = PT.m_hat_from_fx(cov[item, choice[item]])
            assert abs(m_rows[h, 64 * s:64 * s + 64].mean() - m_hat) < 2e-3, (item, ix.cand)
    for h in range(Hq):
        assert abs(m_head[h] - m_rows[h].mean()) < 1e-5
        assert cert_head[h, 1] >= 0
    return layer, choice


def test_pipeline_small_layer_with_segments():
    cands = [C(PT.A_SHAPE, 8, 128), C(PT.A_SHAPE, 8, 256), C(PT.VERTICAL_SLASH, 32, 48), C(PT.VERTICAL_SLASH, 64, 96),
             C(PT.BLOCK_SPARSE, 3), C(PT.BLOCK_SPARSE, 6), C(PT.DENSE)]
    cfg = rs.RouteConfig(budget_frac=0.45, cert_max=0.6)
    layer, choice = run_and_check(tiny_spec(61, 1536, 4, 2), [0, 768, 1536], cands, cfg, "small")
    assert len(set(choice.tolist())) > 1          # the router really mixes patterns on this input


def test_pipeline_tight_budget_and_abs_certificate():
    cands = [C(PT.A_SHAPE, 8, 128), C(PT.VERTICAL_SLASH, 32, 48), C(PT.BLOCK_SPARSE, 3), C(PT.DENSE)]
    cfg = rs.RouteConfig(budget_frac=0.2, cert_max=0.05, cert_mode=rs.RS_CERT_ABS, expand_first=False)
    run_and_check(tiny_spec(63, 1024, 4, 4), [0, 1024], cands, cfg, "abs")


def test_config1_single_head_vertical_slash():
    """n = 4096, one head, vertical-slash (256 verticals, 512 slashes) forced through a two-entry library."""
    spec = config1_spec(toeplitz=True)
    cands = [C(PT.VERTICAL_SLASH, 256, 512), C(PT.DENSE)]
    cfg = rs.RouteConfig(budget_frac=0.6, cert_max=None)
    layer, choice = run_and_check(spec, [0, 4096], cands, cfg, "config1")
    assert choice.tolist() == [0]


def test_profiled_cost_table_routes_like_the_oracle():
    """Measured kernel times as the router's cost table (hardware profiling of Section 3.1 / 3.5): the device
    decision equals the oracle's on the same table."""
    cands = [C(PT.A_SHAPE, 8, 128), C(PT.VERTICAL_SLASH, 32, 48), C(PT.BLOCK_SPARSE, 3), C(PT.DENSE)]
    spec = tiny_spec(71, 2048, 4, 2)
    L = make_layer(spec)
    p = rs.Problem(4, 2, 2048)
    layer = rs.RoutedPrefillLayer(p, [(c.pattern, c.b0, c.b1) for c in cands], rs.RouteConfig(budget_frac=0.5, cert_max=0.9))
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    info = layer.profile_costs(Q, K, V, reps=2)
    table = layer.cost_table.cpu().numpy()
    assert table.shape == (4, 4) and np.all(table >= 1) and len(info["candidate_ms"]) == 4
    assert abs(table.sum(axis=0)[3] - info["candidate_ms"][3] * 1e6) <= 4          # shares add up to the measured time
    layer.forward(Q, K, V)
    rs.check_status(layer.status, "profiled")
    stats = layer.stats.cpu().numpy()
    vmax = layer.vmax.cpu().numpy()
    want, _ = RT.route(cands, stats[:, :, :4].astype(np.uint64), table, np.array([vmax[0, h // 2] for h in range(4)], np.float32),
                       RT.RouteParams(budget=layer.cost_budget, t_probe=layer.cost_t_probe, cert_max=0.9))
    assert np.array_equal(layer.choice.cpu().numpy(), want)


@pytest.mark.parametrize("online", [True, False])
def test_split_launches_give_the_single_launch_result(online):
    """Launch ablation: one launch per KV group / per head computes exactly what the single launch computes."""
    n, Hq, Hkv = 1152, 8, 2
    L = make_layer(tiny_spec(91, n, Hq, Hkv))
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    p = rs.Problem(Hq, Hkv, n)
    lib = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_VERTICAL_SLASH, 48, 160), (rs.RS_VERTICAL_SLASH, 96, 320),
           (rs.RS_BLOCK_SPARSE, 4, 0), (rs.RS_DENSE, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=0.5, cert_max=None))
    if online:
        layer.forward(Q, K, V)
    else:                                              # every pattern present, index arrays in the materialised layout
        fixed = torch.tensor([0, 1, 2, 3, 4, 3, 2, 1], dtype=torch.int32, device="cuda")
        layer.forward(Q, K, V, fixed_choice=fixed)
    rs.check_status(layer.status, "single launch")
    want_O, want_lse = layer.O.clone(), layer.lse_sel.clone()
    for heads in (Hq // Hkv, 1):
        layer.O.zero_(); layer.lse_sel.zero_()
        layer.attention_split(Q, K, V, heads)
        rs.check_status(layer.status, "split launches")
        assert torch.equal(layer.O, want_O) and torch.equal(layer.lse_sel, want_lse), heads


def test_layer_replays_from_a_cuda_graph():
    """The whole layer pass (probe, evaluation, routing on the device, materialisation, attention, certificate; the
    side-stream fork / join inside the probe and index calls included) can be captured once and replayed: no host
    decision sits between the steps."""
    n, Hq, Hkv = 1024, 4, 2
    L = make_layer(tiny_spec(93, n, Hq, Hkv))
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    p = rs.Problem(Hq, Hkv, n, [0, 384, 1024])
    lib = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_VERTICAL_SLASH, 48, 160), (rs.RS_BLOCK_SPARSE, 4, 0), (rs.RS_DENSE, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=0.5, cert_max=0.6))
    layer.forward(Q, K, V)                              # eager: also does the one-time kernel attribute set-up
    torch.cuda.synchronize()
    rs.check_status(layer.status, "eager layer")
    want_O, want_choice, want_m = layer.O.clone(), layer.choice.clone(), layer.m_head.clone()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        layer.forward(Q, K, V)
    for other_seed in (94, 93):                         # new inputs in the same buffers, then the first ones again
        L2 = make_layer(tiny_spec(other_seed, n, Hq, Hkv))
        Q.copy_(dev_bf16(L2["Q"])); K.copy_(dev_bf16(L2["K"])); V.copy_(dev_bf16(L2["V"]))
        layer.O.zero_(); layer.choice.fill_(-1)
        g.replay()
        torch.cuda.synchronize()
        rs.check_status(layer.status, "replayed layer")
    assert torch.equal(layer.choice, want_choice) and torch.equal(layer.O, want_O) and torch.equal(layer.m_head, want_m)


def test_streamed_host_passes_match_the_plain_call():
    """Overlapped host-buffer passes (StreamedPrefill) return, for every pass, what the plain call returns."""
    n, Hq, Hkv = 1024, 4, 2
    p = rs.Problem(Hq, Hkv, n)
    lib = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_VERTICAL_SLASH, 48, 160), (rs.RS_BLOCK_SPARSE, 4, 0), (rs.RS_DENSE, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=0.4, cert_max=0.5))
    hosts, want = [], []
    for seed in (71, 72, 73, 74, 75):
        L = make_layer(tiny_spec(seed, n, Hq, Hkv))
        Qh, Kh, Vh = (torch.from_numpy(L[k].view(np.int16)).view(torch.bfloat16).pin_memory() for k in ("Q", "K", "V"))
        hosts.append((Qh, Kh, Vh, torch.zeros((Hq, n, 128), dtype=torch.bfloat16).pin_memory()))
        layer.forward(Qh.cuda(), Kh.cuda(), Vh.cuda())
        torch.cuda.synchronize()
        want.append(layer.O.cpu().clone())
    pipe = rs.StreamedPrefill(layer)
    for Qh, Kh, Vh, Oh in hosts:
        pipe.submit(Qh, Kh, Vh, Oh)
    pipe.finish()
    torch.cuda.synchronize()
    rs.check_status(layer.status, "streamed passes")
    for k, (_, _, _, Oh) in enumerate(hosts):
        assert torch.equal(Oh, want[k]), k


def test_budgets_larger_than_the_sequence():
    """One 64-row block with vertical-slash budgets beyond the number of keys: the lists are clamped to the keys that exist."""
    cands = [C(PT.VERTICAL_SLASH, 8, 139), C(PT.VERTICAL_SLASH, 119, 140), C(PT.BLOCK_SPARSE, 4), C(PT.DENSE)]
    run_and_check(tiny_spec(80, 64, 4, 2), [0, 64], cands, rs.RouteConfig(budget_frac=0.6, cert_max=0.8), "one block")


def _random_case(seed):
    """Random geometry, segments, candidate library and router settings for the stage-by-stage comparison."""
    rng = np.random.default_rng(seed)
    Hkv = int(rng.choice([1, 2, 4]))
    Hq = Hkv * int(rng.choice([1, 2, 4]))
    nb = int(rng.integers(1, 24))
    n_seg = int(rng.integers(1, min(4, nb) + 1))
    cuts = sorted(rng.choice(np.arange(1, nb), size=n_seg - 1, replace=False).tolist()) if n_seg > 1 else []
    bounds = [0] + [64 * c for c in cuts] + [64 * nb]
    cands = [C(PT.A_SHAPE, int(rng.integers(0, 100)), int(rng.integers(1, 400))) for _ in range(int(rng.integers(0, 3)))]
    cands.sort(key=lambda c: c.b0 + c.b1)
    # candidate evaluation needs sink and window disjoint on the probe rows of every segment
    cands = [c for c in cands if all(c.b1 >= q1 or q1 - 64 - c.b1 + 1 >= c.b0 for q1 in bounds[1:])]
    kv = ks = 0
    for a, b in sorted((int(rng.integers(1, 200)), int(rng.integers(1, 300))) for _ in range(int(rng.integers(0, 4)))):
        kv, ks = max(kv + 1, a), max(ks + 1, b)           # budgets nested inside the family
        cands.append(C(PT.VERTICAL_SLASH, kv, ks))
    for kb in sorted(set(int(x) for x in rng.integers(1, 12, size=int(rng.integers(0, 3))))):
        cands.append(C(PT.BLOCK_SPARSE, kb))
    cands.append(C(PT.DENSE))
    cfg = rs.RouteConfig(budget_frac=float(rng.uniform(0.05, 0.9)), alpha=float(rng.choice([0.0, 1.0, 2.5])),
                         delta_q=float(rng.choice([0.0, 0.02])), cert_max=[None, 0.05, 0.3, 0.8][int(rng.integers(0, 4))],
                         cert_mode=int(rng.choice([rs.RS_CERT_REL, rs.RS_CERT_ABS])), expand_first=bool(rng.integers(0, 2)))
    spec = tiny_spec(1000 + seed, 64 * nb, Hq, Hkv, toeplitz=bool(rng.integers(0, 2)), n_vert=int(rng.integers(0, 6)))
    return spec, bounds, cands, cfg


@pytest.mark.parametrize("seed", range(24))
def test_random_small_layers(seed):
    """Seeded random cases of the whole path (ragged segment lengths, one-block segments, budgets beyond the segment,
    libraries without some family, every router setting), each checked stage by stage like the fixed cases above."""
    spec, bounds, cands, cfg = _random_case(seed)
    run_and_check(spec, bounds, cands, cfg, f"random {seed}")


@pytest.mark.parametrize("online", [True, False])
def test_one_call_layer_equals_the_staged_calls(online):
    """rs_routed_prefill_layer enqueues the same seven calls the staged path issues one by one: every output is
    bit-identical, with online routing and with given routes."""
    n, Hq, Hkv = 1280, 8, 2
    L = make_layer(tiny_spec(73, n, Hq, Hkv))
    p = rs.Problem(Hq, Hkv, n, [0, 512, 1280])
    cands = [(rs.RS_A_SHAPE, 8, 128), (rs.RS_VERTICAL_SLASH, 32, 48), (rs.RS_VERTICAL_SLASH, 64, 96),
             (rs.RS_BLOCK_SPARSE, 3, 0), (rs.RS_BLOCK_SPARSE, 6, 0), (rs.RS_DENSE, 0, 0)]
    Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
    fixed = None if online else torch.tensor([i % len(cands) for i in range(p.n_items)], dtype=torch.int32, device="cuda")
    outs = []
    for one_call in (False, True):
        layer = rs.RoutedPrefillLayer(p, cands, rs.RouteConfig(budget_frac=0.4, cert_max=0.5))
        layer.one_call = one_call
        layer.forward(Q, K, V, fixed_choice=fixed)
        rs.check_status(layer.status, f"one_call={one_call}")
        outs.append([t.clone() for t in (layer.O, layer.lse_sel, layer.onorm, layer.choice, layer.m_row, layer.m_head,
                                         layer.cert_head, layer.counters)] + ([layer.stats.clone(), layer.report.clone()] if online else []))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    if online:
        assert len(set(outs[0][3].tolist())) > 1


def test_graphed_prefill_replays_with_new_inputs():
    """GraphedPrefill: inputs handed to run() are copied into the captured buffers; every replay routes anew and gives
    what the plain call gives."""
    n, Hq, Hkv = 768, 4, 2
    p = rs.Problem(Hq, Hkv, n)
    lib = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_VERTICAL_SLASH, 48, 160), (rs.RS_BLOCK_SPARSE, 4, 0), (rs.RS_DENSE, 0, 0)]
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=0.5, cert_max=0.6))
    ref = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(budget_frac=0.5, cert_max=0.6))
    L0 = make_layer(tiny_spec(201, n, Hq, Hkv))
    gp = rs.GraphedPrefill(layer, dev_bf16(L0["Q"]), dev_bf16(L0["K"]), dev_bf16(L0["V"]))
    for seed in (202, 203, 201):
        L = make_layer(tiny_spec(seed, n, Hq, Hkv))
        Q, K, V = dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])
        O = gp.run(Q, K, V)
        want = ref.forward(Q, K, V)
        torch.cuda.synchronize()
        rs.check_status(layer.status, f"replay {seed}")
        assert torch.equal(O, want) and torch.equal(layer.choice, ref.choice) and torch.equal(layer.m_head, ref.m_head)


def test_two_layers_on_two_streams():
    """Two layers issued from two streams at the same time share the library's per-device side stream (forked from and
    joined into each caller's stream with events): both get what they get when they run alone."""
    n, Hq, Hkv = 1024, 4, 2
    p = rs.Problem(Hq, Hkv, n, [0, 448, 1024])
    lib = [(rs.RS_A_SHAPE, 64, 128), (rs.RS_VERTICAL_SLASH, 48, 160), (rs.RS_BLOCK_SPARSE, 4, 0), (rs.RS_DENSE, 0, 0)]
    cfg = rs.RouteConfig(budget_frac=0.5, cert_max=0.6)
    data = []
    for seed in (301, 302):
        L = make_layer(tiny_spec(seed, n, Hq, Hkv))
        data.append((dev_bf16(L["Q"]), dev_bf16(L["K"]), dev_bf16(L["V"])))
    want = []
    for Q, K, V in data:
        layer = rs.RoutedPrefillLayer(p, lib, cfg)
        layer.forward(Q, K, V)
        torch.cuda.synchronize()
        want.append((layer.O.clone(), layer.choice.clone(), layer.lse_sel.clone()))
    layers = [rs.RoutedPrefillLayer(p, lib, cfg) for _ in range(2)]
    streams = [torch.cuda.Stream() for _ in range(2)]
    torch.cuda.synchronize()
    for rep in range(4):
        for k in range(2):
            with torch.cuda.stream(streams[k]):
                layers[k].forward(*data[k])
    torch.cuda.synchronize()
    for k in range(2):
        rs.check_status(layers[k].status, f"stream {k}")
        assert torch.equal(layers[k].O, want[k][0]) and torch.equal(layers[k].choice, want[k][1])
        assert torch.equal(layers[k].lse_sel, want[k][2])
