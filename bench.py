#!/usr/bin/env python
"""Benchmark of the routed sparse prefill attention layer (one JSON line on stdout).

A step is one pass of the whole hot path over one layer: probe -> candidate evaluation -> routing ->
materialisation -> one sparse attention launch -> certificate.  Default workload: the Llama-3.1-8B-shaped
layer (32 query heads, 8 KV heads, d = 128) at n = 131072 with routing decided online (budget 15 % of the
dense FLOPs, relative certificate threshold 0.05), synthetic seeded inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config3|config2|config1] [--n N]
  python bench.py --impl reference ...        # times the CPU oracle on the host cores instead

Multi-GPU: the path has no exchange step, so N ranks run N independent replicas of the layer (weak scaling);
the only cross-rank traffic is the barrier and the max-over-ranks of the measured time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


# ----------------------------------------------------------------------------------------- workloads
def workload_spec(name: str, n_override: int | None):
    from synth import config1_spec, config2_spec, config3_spec, config4_layer_spec
    if name == "config4":
        spec = config4_layer_spec(0, n=n_override or 131072, seg_len=(n_override or 131072) // 4)
        return spec, None, dict(budget_frac=0.15, cert_max=0.05), None
    if name == "config1":
        spec = config1_spec(toeplitz=True, n=n_override or 4096)
        lib = [(2, 256, 512), (0, 0, 0)]
        route = dict(budget_frac=0.6, cert_max=None)
        fixed = None
    elif name == "config2":
        spec = config2_spec(n=n_override or 32768)
        lib = [(1, 128, 1024), (2, 1000, 6096), (3, 100, 0), (0, 0, 0)]
        route = dict(budget_frac=1.0, cert_max=None)
        fixed = "seeded 30/30/30/10"
    else:
        spec = config3_spec(n=n_override or 131072)
        lib = None     # 13-candidate default library
        route = dict(budget_frac=0.15, cert_max=0.05)
        fixed = None
    return spec, lib, route, fixed


def fixed_choice_for(lib, n_q_heads):
    from synth import fixed_routes_config2
    pat = fixed_routes_config2(n_q_heads)
    index_of = {c[0]: i for i, c in enumerate(lib)}
    return np.array([index_of[int(x)] for x in pat], dtype=np.int32)


# ----------------------------------------------------------------------------------------- measured DRAM traffic
def measured_traffic(workload: str, n: int, plain: bool):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu capture recorded
    in profiles/dram_traffic.json (null for workloads and router settings that were not captured)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not plain or not os.path.exists(path):
        return None, None
    with open(path) as f:
        table = json.load(f)
    rec = table.get(f"{workload}:n={n}")
    if rec is None:
        return None, None
    return float(rec["dram_bytes_read"]) + float(rec["dram_bytes_write"]), rec.get("how")


# ----------------------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7 or not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------- rank plumbing
def init_ranks(n_gpus: int, backend: str = "nccl"):
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def aggregate_over_ranks(ms_local: float, units_local: float, device=None):
    """Max of the time and sum of the processed units over all ranks (replicas: no data-path collective)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ----------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(L, spec, cands, choice, sets_fn, gpu_O=None, budget_s: float = 20.0, n_heads: int = 8, n_blocks: int = 20,
                  routes: str = "under the routes and index lists the GPU pass chose for this layer"):
    """Times the oracle's masked attention on sampled query blocks under the routed masks.

    Returns (effective TFLOP/s, description, cores, max abs difference to gpu_O on the sampled rows).
    """
    from oracle import attention as OA
    from oracle import patterns as PT
    from synth import bf16_bits_to_f64
    G = spec.n_q_heads // spec.n_kv_heads
    nb = spec.n // 64
    heads = sorted(set(int(h) for h in np.linspace(0, spec.n_q_heads - 1, n_heads)))
    blocks = sorted(set(int(b) for b in np.linspace(nb // 16, nb - 1, n_blocks)))
    t_used, pairs_done, rows_done, worst = 0.0, 0, 0, 0.0
    kv_cache = {}
    for h in heads:
        g = h // G
        if g not in kv_cache:
            kv_cache = {g: (bf16_bits_to_f64(L["K"][g]), bf16_bits_to_f64(L["V"][g]))}
        Kf, Vf = kv_cache[g]
        Qf = bf16_bits_to_f64(L["Q"][h])
        ix = sets_fn(h)
        for qb in blocks:
            if t_used > budget_s:
                break
            rows = np.arange(qb * 64, qb * 64 + 64)
            t0 = time.perf_counter()
            Om, _, _ = OA.masked_attention(Qf, Kf, Vf, lambda r, nk: PT.mask_rows(ix, r, nk), rows, chunk=64)
            t_used += time.perf_counter() - t0
            M = PT.mask_rows(ix, rows, int(rows.max()) + 1) & (np.arange(int(rows.max()) + 1)[None, :] <= rows[:, None])
            pairs_done += int(M.sum())
            rows_done += 64
            if gpu_O is not None:
                worst = max(worst, float(np.abs(gpu_O[h, rows].astype(np.float64) - Om).max()))
    tflops = 512.0 * pairs_done / max(t_used, 1e-9) / 1e12
    desc = (f"oracle masked attention on {rows_done} sampled query rows (heads {heads}, query blocks {blocks}) of the "
            f"same layer {routes}, {t_used:.1f} s; effective = 512 FLOP x selected pairs / time")
    return tflops, desc, os.cpu_count(), worst


def download_sets(layer, cands, choice):
    """Device index lists of the routed candidates -> the oracle's IndexSet objects (CPU-baseline leg only)."""
    from oracle import patterns as PT
    sets = []
    for item, d in enumerate(layer.download_index_lists(choice)):
        ix = PT.IndexSet(cand=cands[choice[item]], q0=d["q0"], q1=d["q1"])
        for name in ("V", "S", "D", "blk"):
            if name in d:
                setattr(ix, name, d[name])
        sets.append(ix)
    return sets


# ----------------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config3", choices=["config1", "config2", "config3", "config4"])
    ap.add_argument("--layers", type=int, default=32, help="config4: layers of the attention-only stack per step")
    ap.add_argument("--distinct-layers", type=int, default=2, help="config4: distinct generated layers that are cycled")
    ap.add_argument("--cost", default="flops", choices=["flops", "measured"],
                    help="router cost table: FLOPs of the selected pairs, or kernel times profiled before the timed region")
    ap.add_argument("--rescue", action="store_true", help="fallback variant: cheapest passing sparse candidate of any family before dense")
    ap.add_argument("--calibration", type=str, default=None,
                    help="JSON written by `python -m paper_2608_29058_b200.calibrate`: installs delta_q and the predictor e")
    ap.add_argument("--beta", type=float, default=0.0, help="weight of the calibrated predictor e in Eq. 4 (needs --calibration)")
    ap.add_argument("--launch-ablation", action="store_true",
                    help="also time the attention stage as one launch per KV group and as one launch per head")
    ap.add_argument("--ablations", action="store_true",
                    help="router ablations of the paper's Table 3 on the config-3 layer, JSONL output")
    ap.add_argument("--mixture", action="store_true",
                    help="u of Eq. 4 = disagreement among the recent / uniform / boundary rows of the query mixture (pooled probe)")
    ap.add_argument("--mixture-lists", action="store_true",
                    help="vertical / slash lists ranked by the query mixture of Eq. 3 at key resolution (four 16-row runs) "
                         "instead of the last 64 rows alone (the paper's 'Recent queries only' ablation is the default)")
    ap.add_argument("--graph", action="store_true",
                    help="also time the layer replayed from a CUDA graph (whole pass captured once; for launch-bound sizes)")
    ap.add_argument("--from-hidden", action="store_true",
                    help="the layer pass with its producer in front: QKV projection + rotary embedding (Llama-3.1-8B "
                         "geometry, seeded weights) with the probe's side outputs fused into its epilogue; --n sets the length")
    ap.add_argument("--sweep", action="store_true", help="config-5 sweep: n x budget x forced-dense cells, JSONL output")
    ap.add_argument("--n", type=int, default=None, help="override the sequence length (smaller profiling case)")
    ap.add_argument("--out-dir", default="bench_out", help="directory for the JSONL files of --sweep and --ablations")
    ap.add_argument("--no-extra", action="store_true",
                    help="config3: skip the two untimed side runs (the literal planted-structure generator at this length, "
                         "and the certificate read in ABS mode)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.from_hidden:
        return from_hidden(args)
    if args.sweep:
        return sweep(args)
    if args.ablations:
        return ablations(args)
    if args.workload == "config4" and args.impl == "ours":
        return stack(args)

    from synth import make_layer
    spec, lib, route_kw, fixed = workload_spec(args.workload, args.n)
    metric = "effective TFLOP/s of routed sparse prefill attention (FLOPs of selected query-key pairs / layer time)"
    generator = {"config1": "planted-structure generator with the task's literal constants (sinks 4, verticals 3, local 0.5)",
                 "config2": "planted-structure generator, per-head random sink / vertical / local strengths",
                 "config3": "archetype generator (local / vertical / topic / diffuse heads), boosts scaled by log(n/4096)"}
    config = {"workload": f"{args.workload}: Hq={spec.n_q_heads} Hkv={spec.n_kv_heads} d=128 n={spec.n}, "
                          + generator.get(args.workload, "") + ", "
                          + ("routes fixed from seed" if fixed else
                             f"online routing, budget {route_kw['budget_frac']:.2f} of dense FLOPs, cert_max {route_kw['cert_max']} "
                             f"with cert_mode=REL (Eq. 5 without the V_max factor)"),
              "l2": "inputs (Q,K,V,O > 126 MB) exceed L2; no explicit flush" if spec.n >= 32768 else "small case, L2 resident",
              "replicas": args.gpus}

    if args.impl == "reference":
        rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
        if rank != 0:
            return 0
        return reference_arm(args, spec, lib, route_kw, fixed, metric, config)

    import torch
    import paper_2608_29058_b200 as rs
    rank, world = init_ranks(args.gpus)
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = measured_peaks()

    L = make_layer(spec)
    to_dev = lambda bits: torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
    Q, K, V = to_dev(L["Q"]), to_dev(L["K"]), to_dev(L["V"])
    p = rs.Problem(spec.n_q_heads, spec.n_kv_heads, spec.n, [int(x) for x in L["seg_bounds"]])
    layer = rs.RoutedPrefillLayer(p, lib, rs.RouteConfig(rescue_any=args.rescue, mixture_u=args.mixture,
                                                           mixture_lists=args.mixture_lists, **route_kw), device=dev)
    risk_calibration = None
    if args.calibration:
        with open(args.calibration) as f:
            calib = json.loads(f.read())
        layer.use_calibration(calib, beta=args.beta)
        risk_calibration = {"file": os.path.basename(args.calibration), "delta_q": calib["delta_q"], "beta": args.beta,
                            "q": calib.get("q"), "calibrated_at_n": calib.get("n")}
    fixed_t = None
    if fixed:
        fixed_t = torch.from_numpy(fixed_choice_for(layer.cands, spec.n_q_heads)).to(dev)

    def step(record=False):
        return layer.forward(Q, K, V, fixed_choice=fixed_t, record_events=record)

    def sync_all():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    rs.check_status(layer.status, "warm-up")
    calibration = None
    if args.cost == "measured" and not fixed:
        # offline hardware profiling of the library (outside the timed region), then the router uses the measured table
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(3):
            step()
        f1.record()
        torch.cuda.synchronize()
        calibration = layer.profile_costs(Q, K, V)
        calibration["flop_routed_ms_per_layer"] = f0.elapsed_time(f1) / 3
        calibration["flop_routed_routes"] = layer.choice.cpu().tolist()
        for _ in range(args.warmup):
            step()
        torch.cuda.synchronize()

    # ---- timed region: K steps, CUDA events on the launching stream, per-stage events inside every step
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stage_events = []
    layer.counters.zero_()
    t_wall0 = time.time()
    e0.record()
    for _ in range(args.steps):
        step(record=True)
        stage_events.append(layer.events)
    e1.record()
    sync_all()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    ms_local = e0.elapsed_time(e1) / args.steps
    rs.check_status(layer.status, "timed region")

    names = ["probe", "evaluate", "route", "materialise", "attention", "certificate"]
    stages = {nm: float(np.mean([ev[i].elapsed_time(ev[i + 1]) for ev in stage_events])) for i, nm in enumerate(names)}
    # medians as well: one slow event pair (a clock change between two stage events) shifts the mean of a 0.01 ms stage
    stages_med = {nm: float(np.median([ev[i].elapsed_time(ev[i + 1]) for ev in stage_events])) for i, nm in enumerate(names)}
    step_ms = [ev[0].elapsed_time(ev[6]) for ev in stage_events]      # per-step device time (first to last stage event)
    step_stats = {"median": float(np.median(step_ms)), "p95": float(np.percentile(step_ms, 95)),
                  "min": float(np.min(step_ms)), "max": float(np.max(step_ms)), "n": len(step_ms)}
    counters = layer.counters.cpu().numpy()
    chunks_per_step = int(counters[0]) // args.steps
    choice = layer.choice.cpu().numpy()
    stats = layer.stats.cpu().numpy()
    if fixed:
        layer.evaluate_candidates()      # pair counts of the fixed routes (outside the timed region)
        torch.cuda.synchronize()
        stats = layer.stats.cpu().numpy()
    pairs_sel = int(sum(int(stats[it, choice[it], 4]) for it in range(p.n_items)))
    f_mask = 512.0 * pairs_sel
    f_tile = chunks_per_step * (128 * 64 * 512.0)
    f_dense = float(rs.dense_flops(p.seg_bounds, p.n_q_heads))

    ms, units = aggregate_over_ranks(ms_local, f_mask, dev)
    value = units / (ms * 1e-3) / 1e12

    # ---- own dense kernel (denominator of the speed-up), same inputs
    dense_ms = None
    if not args.no_dense:
        ws = layer.ws
        lse_d = torch.empty((p.n_q_heads, p.n_keys), dtype=torch.float32, device=dev)
        O_d = torch.empty_like(layer.O)
        reps = 2 if spec.n > 65536 else 3
        rs.rs_dense_prefill_attn(p, Q, K, V, O_d, lse_d, None, None, ws, layer.status)
        torch.cuda.synchronize()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record()
        for _ in range(reps):
            rs.rs_dense_prefill_attn(p, Q, K, V, O_d, lse_d, None, None, ws, layer.status)
        d1.record()
        torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / reps
        del O_d, lse_d

    # ---- the same layer pass through the one-call entry point (no stage events, no Python between the stages)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    o0.record()
    for _ in range(args.steps):
        step()
    o1.record()
    torch.cuda.synchronize()
    rs.check_status(layer.status, "one-call passes")
    one_call_ms = o0.elapsed_time(o1) / args.steps

    # ---- the same layer pass replayed from a CUDA graph (no host work between the launches)
    graph_ms = None
    if args.graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        g.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(args.steps):
            g.replay()
        g1.record()
        torch.cuda.synchronize()
        rs.check_status(layer.status, "graph replay")
        graph_ms = g0.elapsed_time(g1) / args.steps

    # ---- launch ablation (Section 3.4 / Table 3: grouping heads into one launch against per-group / per-head launches)
    launch_ablation = None
    if args.launch_ablation and p.n_segments == 1:
        def timed(fn, reps=3):
            fn()
            torch.cuda.synchronize()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            for _ in range(reps):
                fn()
            a1.record()
            torch.cuda.synchronize()
            return a0.elapsed_time(a1) / reps
        group = p.n_q_heads // p.n_kv_heads
        launch_ablation = {
            "single_launch_ms": timed(lambda: layer.attention(Q, K, V)),
            "per_kv_group_ms": timed(lambda: layer.attention_split(Q, K, V, group)),
            "per_head_ms": timed(lambda: layer.attention_split(Q, K, V, 1)),
            "launches": {"single": 1, "per_kv_group": p.n_kv_heads, "per_head": p.n_q_heads},
            "note": "attention stage only, same routes and index arrays; every launch also runs its own work-list kernels"}

    # ---- end to end through the public call with pinned host buffers
    e2e = None
    if not args.no_e2e:
        Qh, Kh, Vh = (torch.from_numpy(L[k].view(np.int16)).view(torch.bfloat16).pin_memory() for k in ("Q", "K", "V"))
        Oh = torch.empty(tuple(layer.O.shape), dtype=layer.O.dtype).pin_memory()
        bufs = (Q, K, V)
        # Every step copies its Q, K, V from pinned host memory and its O back; the copies of neighbouring steps overlap
        # with the kernels (three streams, two device buffer sets).
        pipe = rs.StreamedPrefill(layer)
        def e2e_step():
            pipe.submit(Qh, Kh, Vh, Oh, fixed_choice=fixed_t)
        e2e_step()
        pipe.finish()
        sync_all()
        k_e2e = max(4, min(args.steps, 20))      # the first copy in and the last copy out are not hidden: short runs show them
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(k_e2e):
            e2e_step()
        pipe.finish()
        g1.record()
        sync_all()
        rs.check_status(layer.status, "end-to-end steps")
        ms_e2e, units_e2e = aggregate_over_ranks(g0.elapsed_time(g1) / k_e2e, f_mask, dev)
        h2d = sum(int(t.numel() * t.element_size()) for t in (Qh, Kh, Vh))
        d2h = int(Oh.numel() * Oh.element_size())
        e2e = {"value": units_e2e / (ms_e2e * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "overlap": "copies of neighbouring steps overlap the kernels (3 streams, 2 buffer sets); every step copies its own inputs and output"}
        del Qh, Kh, Vh, pipe

    if rank != 0:
        return 0

    plain = args.cost == "flops" and not (args.rescue or args.mixture or args.calibration or args.mixture_lists)
    # ---- side runs outside the timed region: what the headline would be under the two literal readings of the task
    extra = None
    if args.workload == "config3" and not args.no_extra and plain:
        extra = side_runs(rs, torch, dev, spec, p, Q, K, V, layer, route_kw, dense_ms)

    # ---- CPU oracle on a bounded sample of the same workload (also a full-size parity spot check)
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import patterns as PT
        cands = [PT.Candidate(c[0], c[1], c[2]) for c in layer.cands]
        sets = download_sets(layer, cands, choice)
        O_host = layer.O.float().cpu().numpy()
        tf, desc, cores, worst = oracle_sample(L, spec, cands, choice, lambda h: sets[(p.n_segments - 1) * p.n_q_heads + h],
                                               O_host)
        cpu = {"value": tf, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": desc,
               "max_abs_diff_vs_gpu_on_sample": worst}

    peak = peaks["bf16_tflops_sustained"]
    traffic, traffic_how = measured_traffic(args.workload, spec.n, plain)
    attn_ms = stages["attention"]
    achieved = f_tile / (attn_ms * 1e-3) / 1e12
    overhead_ms = stages["probe"] + stages["evaluate"] + stages["route"] + stages["materialise"] + stages["certificate"]
    hist = _route_hist(layer, choice)
    any_vs = any(c[0] == 2 for c in layer.cands)
    any_bs = any(c[0] == 3 for c in layer.cands)
    # kernels of this library per layer pass, stage by stage (memsets and torch copies are not counted)
    nb = spec.n // 64
    n_probe = 2 + 1                                       # two passes (K pooled in pass 1; V_max and the last Q block in pass 2); value norms
    n_probe += 2 if (args.mixture_lists and not fixed) else 0          # the probe on the mixture's runs
    if fixed:
        n_eval, n_route = 0, 0
        n_mat = 3 * any_vs + 2 * any_bs                   # keys / select / finish; fused scores / rows
    else:
        n_eval = 1 + (3 if any_vs else 1 + any_bs)        # closed-form stats + pooled scores; keys + block sums, select, finish / BS evaluation (without VS: block sums, BS evaluation)
        n_eval += 1 if (args.mixture_lists and any_vs) else 0          # block sums separate from the ranking keys
        n_eval += 4 if args.mixture else 0                # pooled probe (3) + mixture coverage
        n_eval += (0 if args.mixture else 3) + 1 if (args.calibration and args.beta > 0) else 0   # pooled probe + predictor
        n_route = 1
        n_mat = 2 * any_bs                                # the evaluation's vertical-slash lists are reused
    n_mat += 0 if (args.mixture and not fixed) else int(any_bs)     # queries of the heads routed to block-sparse
    launches_per_step = n_probe + n_eval + n_route + n_mat + 2 + 1  # + preparation (work list, gather), attention + certificate
    out = {
        "metric": metric, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": config,
        "ms_per_layer": ms, "ms_per_step_stats": step_stats, "dense_ms_per_layer": dense_ms,
        "speedup_vs_own_dense": (dense_ms / ms) if dense_ms else None,
        "dense_tflops": (f_dense / (dense_ms * 1e-3) / 1e12) if dense_ms else None,
        "stage_ms": stages, "overhead_over_attention": overhead_ms / attn_ms,
        "stage_ms_median": stages_med,
        "overhead_over_attention_median": (sum(stages_med.values()) - stages_med["attention"]) / stages_med["attention"],
        "flops": {"selected_pairs": f_mask, "issued_tiles": f_tile, "dense": f_dense,
                  "selected_fraction_of_dense": f_mask / f_dense},
        "routes": hist, "route_report": layer.route_report() if not fixed else None,
        "cost_model": args.cost, "calibration": calibration, "risk_calibration": risk_calibration, "launch_ablation": launch_ablation,
        "one_call_ms_per_layer": one_call_ms, "cuda_graph_ms_per_layer": graph_ms,
        "fallback_rescue": bool(args.rescue), "mixture_uncertainty": bool(args.mixture),
        "mixture_lists": bool(args.mixture_lists),
        "roofline": {"kernel": "rs_attn_kernel (one launch, all heads)", "bound": "tensor", "achieved": achieved,
                     "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_source": f"bf16_tflops_sustained, {peaks['source']}",
                     "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                     "traffic": traffic, "traffic_note": traffic_how,
                     "note": "achieved = 512 FLOP x 128 x 64 pairs per issued chunk / attention-call time (CUDA events)"},
        "stage_ms_targets": {"probe": 0.30, "evaluate": 0.35, "at": "n=131072, config3"},
        "extra": extra,
        "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks, "gpu_launches": launches_per_step * args.steps,
    }
    print(json.dumps(out))
    return 0


def _route_hist(layer, choice):
    hist = {}
    for it in range(len(choice)):
        c = layer.cands[choice[it]]
        key = {0: "dense", 1: "a_shape", 2: "vertical_slash", 3: "block_sparse"}[c[0]] + (f"({c[1]},{c[2]})" if c[0] else "")
        hist[key] = hist.get(key, 0) + 1
    return hist


def side_runs(rs, torch, dev, spec, p, Q, K, V, layer, route_kw, dense_ms, reps: int = 3):
    """Two untimed companions of the config-3 headline, so that the JSON line itself shows what the workload choices do:
    (a) the same layer pass with the certificate read in ABS mode (2 (1 - m_low) V_max against cert_max);
    (b) the same online routing on a layer from the planted-structure generator of configs 1-2 (per-head random sink /
        vertical / local strengths, no scaling with n) at this length."""
    def run(lyr, q, k, v):
        for _ in range(2):
            lyr.forward(q, k, v)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            lyr.forward(q, k, v)
        b.record()
        torch.cuda.synchronize()
        rs.check_status(lyr.status, "side run")
        ms = a.elapsed_time(b) / reps
        choice = lyr.choice.cpu().numpy()
        rep = lyr.route_report()
        return {"ms_per_layer": ms, "speedup_vs_own_dense": (dense_ms / ms) if dense_ms else None,
                "routes": _route_hist(lyr, choice), "fallback_rate": rep["n_fallback"] / p.n_items,
                "dense_items": int(sum(1 for c in choice if lyr.cands[c][0] == 0))}
    out = {}
    saved = layer.cfg.cert_mode
    layer.cfg.cert_mode = rs.RS_CERT_ABS
    out["cert_mode_abs"] = run(layer, Q, K, V)
    out["cert_mode_abs"]["note"] = "same layer and budget; fallback test 2 (1 - m_low) V_max > cert_max"
    layer.cfg.cert_mode = saved
    from synth import config2_spec, make_layer
    lit = make_layer(config2_spec(n=spec.n, n_q_heads=spec.n_q_heads, n_kv_heads=spec.n_kv_heads))
    q2, k2, v2 = (_to_dev(lit[k], dev) for k in ("Q", "K", "V"))
    out["literal_generator"] = run(layer, q2, k2, v2)
    out["literal_generator"]["note"] = ("planted-structure generator of configs 1-2 at this length (constants not scaled "
                                        "with n), same budget and REL certificate")
    del q2, k2, v2
    layer.forward(Q, K, V)             # leave the layer holding the headline pass again
    torch.cuda.synchronize()
    return out


def _to_dev(bits, dev):
    import torch
    return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)


def stack(args):
    """Config 4: attention-only prefill stack, per-segment rerouting, one attention launch per layer."""
    import torch
    import paper_2608_29058_b200 as rs
    from synth import config4_layer_spec, make_layer
    rank, world = init_ranks(args.gpus)
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    n = args.n or 131072
    layers = []
    for l in range(max(1, args.distinct_layers)):
        spec = config4_layer_spec(l, n=n, seg_len=n // 4)
        L = make_layer(spec)
        layers.append((spec, _to_dev(L["Q"], dev), _to_dev(L["K"], dev), _to_dev(L["V"], dev)))
    spec0 = layers[0][0]
    p = rs.Problem(spec0.n_q_heads, spec0.n_kv_heads, n, spec0.seg_bounds())
    layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(budget_frac=0.15, cert_max=0.05), device=dev)

    def step(collect=None):
        for l in range(args.layers):
            _, Q, K, V = layers[l % len(layers)]
            layer.forward(Q, K, V)
            if collect is not None:
                collect.append((layer.choice.clone(), layer.stats.clone()))

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    rs.check_status(layer.status, "warm-up")
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    layer.counters.zero_()
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop(t0, time.time())
    ms_step = e0.elapsed_time(e1) / args.steps
    rs.check_status(layer.status, "timed region")
    chunks = int(layer.counters.cpu().numpy()[0]) // args.steps
    info = []
    step(info)                       # one untimed pass to read the routes and pair counts of every layer
    torch.cuda.synchronize()
    names = {0: "dense", 1: "a_shape", 2: "vertical_slash", 3: "block_sparse"}
    kinds = [s.kind for s in spec0.segments]
    pairs, hist = 0, {}
    for l, (choice, stats) in enumerate(info):
        ch, st = choice.cpu().numpy(), stats.cpu().numpy()
        for it in range(p.n_items):
            pairs += int(st[it, ch[it], 4])
            sp = layers[l % len(layers)][0]
            key = sp.segments[it // p.n_q_heads].kind + ":" + names[layer.cands[ch[it]][0]]
            hist[key] = hist.get(key, 0) + 1
    f_mask, f_tile = 512.0 * pairs, chunks * (128 * 64 * 512.0)
    f_dense = float(rs.dense_flops(p.seg_bounds, p.n_q_heads)) * args.layers
    ms, units = aggregate_over_ranks(ms_step, f_mask, dev)
    if rank != 0:
        return 0
    peaks = measured_peaks()
    out = {"metric": "effective TFLOP/s of routed sparse prefill attention (FLOPs of selected query-key pairs / stack time)",
           "value": units / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "bf16", "data": "synthetic",
           "config": {"workload": f"config4: {args.layers}-layer attention-only stack, Hq=32 Hkv=8 d=128 n={n}, four segments of "
                                  f"{n // 4} with local / delimiter / needle / diffuse structure (order seeded per layer), per-segment "
                                  f"online routing; {len(layers)} distinct generated layers cycled", "replicas": args.gpus,
                      "l2": "inputs exceed L2"},
           "ms_per_layer": ms / args.layers, "segment_kinds_layer0": kinds, "routes_by_segment_kind": hist,
           "flops": {"selected_pairs": f_mask, "issued_tiles": f_tile, "dense": f_dense,
                     "selected_fraction_of_dense": f_mask / f_dense},
           "roofline": {"kernel": "whole stack (attention dominates)", "bound": "tensor",
                        "achieved": f_tile / (ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                        "frac": f_tile / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                        "peak_source": f"bf16_tflops_sustained, {peaks['source']}", "traffic": None},
           "clocks": clocks, "gpu_launches": 14 * args.layers * args.steps}
    print(json.dumps(out))
    return 0


def from_hidden(args):
    """Projection-fused layer pass (Section 3.4: the probe as a reduction beside the projection kernels).  X and W are
    seeded Gaussians (no structure is planted, so the router sends most heads to dense); what is measured is the
    producer itself and what its fused side outputs take off the probe."""
    import torch
    import paper_2608_29058_b200 as rs
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n = args.n or 16384
    dm, Hq, Hkv = 4096, 32, 8
    gen = torch.Generator(device=dev).manual_seed(260829058)
    X = torch.randn((n, dm), generator=gen, device=dev).to(torch.bfloat16)
    W = (torch.randn(((Hq + 2 * Hkv) * 128, dm), generator=gen, device=dev) / dm ** 0.5).to(torch.bfloat16)
    inv = 500000.0 ** (-torch.arange(0, 128, 2, device=dev, dtype=torch.float64) / 128)
    ang = torch.arange(n, device=dev, dtype=torch.float64)[:, None] * inv[None, :]
    cos, sin = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    p = rs.Problem(Hq, Hkv, n)
    layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(budget_frac=0.15, cert_max=0.05), device=dev)
    for _ in range(max(3, args.warmup)):
        layer.forward_from_hidden(X, W, cos, sin)
    torch.cuda.synchronize()
    rs.check_status(layer.status, "warm-up")
    evs = []
    for _ in range(args.steps):
        layer.forward_from_hidden(X, W, cos, sin, record_events=True)
        evs.append(layer.events_hidden)
    torch.cuda.synchronize()
    rs.check_status(layer.status, "timed region")
    names = ["projection", "probe", "evaluate", "route", "materialise", "attention", "certificate"]
    st = {nm: float(np.median([e[i].elapsed_time(e[i + 1]) for e in evs])) for i, nm in enumerate(names)}
    # the same tensors through the ordinary pass (the probe pools by itself): what the fusion takes off the probe
    Q, K, V = layer._qkv
    plain = []
    for _ in range(args.steps):
        layer.forward(Q, K, V, record_events=True)
        plain.append(layer.events)
    torch.cuda.synchronize()
    probe_plain = float(np.median([e[0].elapsed_time(e[1]) for e in plain]))
    flops = 2.0 * n * dm * (Hq + 2 * Hkv) * 128
    peaks = measured_peaks()
    tf = flops / (st["projection"] * 1e-3) / 1e12
    print(json.dumps({"metric": "QKV projection + rotary embedding with fused probe side outputs, then the routed layer pass",
                      "config": {"workload": f"from hidden states: d_model=4096 Hq=32 Hkv=8 d=128 n={n}, seeded Gaussian X and W"},
                      "stage_ms_median": st, "projection_tflops": tf,
                      "projection_frac_of_burst_peak": tf / peaks["bf16_tflops"], "peak_source": peaks["source"],
                      "probe_ms_when_it_pools_itself": probe_plain, "probe_ms_fed_by_projection": st["probe"],
                      "steps": args.steps, "data": "synthetic", "dtype": "bf16"}))
    return 0


def ablations(args):
    """The router ablations of the paper's Table 3, on the config-3 layer: time per layer, fallback rate, share of the
    dense pairs computed and, in place of task scores (no model, no datasets here), the exactly retained attention mass
    on the audited probe rows: mean over heads, mean of the worst tenth of the heads, minimum."""
    import torch
    import paper_2608_29058_b200 as rs
    from synth import config3_spec, make_layer
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n = args.n or 131072
    out_dir = os.path.abspath(args.out_dir)
    os.makedirs(out_dir, exist_ok=True)
    path = os.path.join(out_dir, f"ablations_config3_n{n}.jsonl")
    spec = config3_spec(n)
    L = make_layer(spec)
    Q, K, V = _to_dev(L["Q"], dev), _to_dev(L["K"], dev), _to_dev(L["V"], dev)
    p = rs.Problem(spec.n_q_heads, spec.n_kv_heads, n)
    full_lib = rs.default_library()
    one_budget = [full_lib[1], full_lib[5], full_lib[9], full_lib[12]]     # second budget of each family + dense
    base = dict(budget_frac=0.15, cert_max=0.05)
    # routes of another input of the same recipe, applied unchanged ("no input routing")
    Lc = make_layer(config3_spec(n, seed_offset=5000))
    cal_layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(**base), device=dev)
    cal_layer.forward(_to_dev(Lc["Q"], dev), _to_dev(Lc["K"], dev), _to_dev(Lc["V"], dev))
    static_routes = cal_layer.choice.clone()
    del cal_layer, Lc
    variants = [
        ("full", None, rs.RouteConfig(**base), {}),
        ("no input routing (routes of another input)", None, rs.RouteConfig(**base), {"fixed": static_routes}),
        ("no uncertainty score (alpha = 0)", None, rs.RouteConfig(alpha=0.0, **base), {}),
        ("no dense fallback", None, rs.RouteConfig(budget_frac=0.15, cert_max=None), {}),
        ("one fixed budget per family", one_budget, rs.RouteConfig(**base), {}),
        ("profiled latency table instead of FLOPs", None, rs.RouteConfig(**base), {"measured": True}),
        ("per-head launches", None, rs.RouteConfig(**base), {"per_head": True}),
        ("fallback rescue (any family before dense)", None, rs.RouteConfig(rescue_any=True, **base), {}),
        ("greedy back-fill of leftover budget", None, rs.RouteConfig(backfill=True, **base), {}),
        ("uncertainty from recent / uniform / boundary rows (query mixture)", None, rs.RouteConfig(mixture_u=True, **base), {}),
        ("the same with alpha = 4", None, rs.RouteConfig(mixture_u=True, alpha=4.0, **base), {}),
        ("lists ranked by the query mixture (four 16-row runs) instead of the recent rows only", None,
         rs.RouteConfig(mixture_lists=True, **base), {}),
        ("layer-level router: one candidate for all heads", None, rs.RouteConfig(global_pattern=True, **base), {}),
        ("layer-level router without fallback", None, rs.RouteConfig(global_pattern=True, budget_frac=0.15, cert_max=None), {}),
    ]
    rows = []
    with open(path, "w") as f:
        for name, lib, cfg, opt in variants:
            layer = rs.RoutedPrefillLayer(p, lib, cfg, device=dev)
            fixed = opt.get("fixed")
            if opt.get("measured"):
                layer.forward(Q, K, V)
                layer.profile_costs(Q, K, V)
            for _ in range(2):
                layer.forward(Q, K, V, fixed_choice=fixed)
            torch.cuda.synchronize()
            k = 3
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(k):
                layer.forward(Q, K, V, fixed_choice=fixed, record_events=True)
            e1.record()
            torch.cuda.synchronize()
            rs.check_status(layer.status, name)
            ms = e0.elapsed_time(e1) / k
            st = layer.stage_ms()
            if opt.get("per_head"):
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                layer.attention_split(Q, K, V, 1)
                a0.record()
                for _ in range(k):
                    layer.attention_split(Q, K, V, 1)
                a1.record()
                torch.cuda.synchronize()
                ms = ms - st["attention"] + a0.elapsed_time(a1) / k
            choice = layer.choice.cpu().numpy()
            m_head = np.sort(layer.m_head.cpu().numpy().astype(np.float64))
            worst = max(1, len(m_head) // 10)
            pairs = layer.stats.cpu().numpy()[:, :, 4]
            dense_c = [i for i, c in enumerate(layer.cands) if c[0] == rs.RS_DENSE][0]
            if fixed is None and (pairs.sum() > 0):
                frac = float(sum(pairs[i, choice[i]] for i in range(p.n_items)) / pairs[:, dense_c].sum())
            else:
                frac = None
            rep = layer.route_report() if fixed is None else {"n_fallback": 0}
            row = {"variant": name, "n": n, "ms_per_layer": ms, "fallback_pct": 100.0 * rep["n_fallback"] / p.n_items,
                   "dense_heads": int((choice == dense_c).sum()), "pairs_fraction_of_dense": frac,
                   "retained_mass_mean": float(m_head.mean()), "retained_mass_worst_decile": float(m_head[:worst].mean()),
                   "retained_mass_min": float(m_head[0]), "stage_ms": st}
            f.write(json.dumps(row) + "\n")
            f.flush()
            rows.append(row)
            del layer
            torch.cuda.empty_cache()
    print(json.dumps({"ablations": [{k: r[k] for k in ("variant", "ms_per_layer", "fallback_pct", "dense_heads",
                                                       "retained_mass_mean", "retained_mass_worst_decile")} for r in rows],
                      "file": path}))
    return 0


def sweep(args):
    """Config 5: n x latency budget x forced-dense fraction on the config-3 layer; one JSON line per cell (resumable)."""
    import torch
    import paper_2608_29058_b200 as rs
    from synth import config3_spec, make_layer
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    out_dir = os.path.abspath(args.out_dir)
    os.makedirs(out_dir, exist_ok=True)
    path = os.path.join(out_dir, "sweep_config5.jsonl")
    done = set()
    if os.path.exists(path):
        for line in open(path):
            try:
                d = json.loads(line)
                done.add((d["n"], d["budget"], d["forced_dense"]))
            except Exception:
                pass
    peaks = measured_peaks()
    ns = [args.n] if args.n else [16384, 32768, 65536, 131072]
    cells = []
    for n in ns:
        spec = config3_spec(n)
        L = make_layer(spec)
        Q, K, V = _to_dev(L["Q"], dev), _to_dev(L["K"], dev), _to_dev(L["V"], dev)
        p = rs.Problem(spec.n_q_heads, spec.n_kv_heads, n)
        layer = rs.RoutedPrefillLayer(p, None, rs.RouteConfig(), device=dev)
        lse_d = torch.empty((p.n_q_heads, n), dtype=torch.float32, device=dev)
        O_d = torch.empty_like(layer.O)
        for _ in range(2):
            rs.rs_dense_prefill_attn(p, Q, K, V, O_d, lse_d, None, None, layer.ws, layer.status)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record()
        for _ in range(2):
            rs.rs_dense_prefill_attn(p, Q, K, V, O_d, lse_d, None, None, layer.ws, layer.status)
        d1.record()
        torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / 2
        del O_d, lse_d
        perm = np.random.default_rng(260829058 + 5).permutation(p.n_q_heads)
        for budget in (0.05, 0.10, 0.20, 0.40):
            for forced in (0.0, 0.25, 0.5, 1.0):
                if (n, budget, forced) in done:
                    continue
                layer.cfg.budget_frac = budget
                fd = torch.zeros(p.n_items, dtype=torch.int32, device=dev)
                fd[torch.from_numpy(perm[:int(round(forced * p.n_q_heads))].copy()).to(dev)] = 1
                for _ in range(max(1, min(args.warmup, 2))):
                    layer.forward(Q, K, V, forced_dense=fd)
                torch.cuda.synchronize()
                layer.counters.zero_()
                k = max(2, min(args.steps, 3))
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(k):
                    layer.forward(Q, K, V, forced_dense=fd, record_events=True)
                e1.record()
                torch.cuda.synchronize()
                rs.check_status(layer.status, "sweep cell")
                ms = e0.elapsed_time(e1) / k
                stages = layer.stage_ms()
                ch, st = layer.choice.cpu().numpy(), layer.stats.cpu().numpy()
                pairs = int(sum(int(st[it, ch[it], 4]) for it in range(p.n_items)))
                f_mask = 512.0 * pairs
                f_tile = int(layer.counters.cpu().numpy()[0]) // k * (128 * 64 * 512.0)
                cell = {"n": n, "budget": budget, "forced_dense": forced, "ms_per_layer": ms, "dense_ms_per_layer": dense_ms,
                        "speedup_vs_own_dense": dense_ms / ms, "effective_tflops": f_mask / (ms * 1e-3) / 1e12,
                        "attention_ms": stages["attention"], "overhead_ms": ms - stages["attention"],
                        "tile_tflops": f_tile / (stages["attention"] * 1e-3) / 1e12,
                        "roofline_frac": f_tile / (stages["attention"] * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                        "selected_fraction_of_dense": f_mask / float(rs.dense_flops(p.seg_bounds, p.n_q_heads)),
                        "n_dense_heads": int(sum(1 for it in range(p.n_items) if layer.cands[ch[it]][0] == 0))}
                with open(path, "a") as f:
                    f.write(json.dumps(cell) + "\n")
                cells.append(cell)
        del layer, Q, K, V
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "config-5 sweep", "cells_run": len(cells), "cells_file": path,
                      "peak": peaks["bf16_tflops_sustained"], "data": "synthetic"}))
    return 0


def reference_arm(args, spec, lib, route_kw, fixed, metric, config):
    """The oracle as it stands, timed on the host cores on a bounded sample of the same workload per step."""
    from synth import make_layer
    from oracle import patterns as PT
    from oracle import probe as OP
    from synth import bf16_bits_to_f64
    import paper_2608_29058_b200.pipeline as pl     # library list only (host data, no GPU work)
    cands_raw = lib if lib is not None else pl.default_library()
    cands = [PT.Candidate(c[0], c[1], c[2]) for c in cands_raw]
    heads = sorted(set(int(h) for h in np.linspace(0, spec.n_q_heads - 1, 4)))
    L = make_layer(spec, heads=heads)
    Lq = {"Q": {h: L["Q"][i] for i, h in enumerate(heads)}, "K": L["K"], "V": L["V"]}
    G = spec.n_q_heads // spec.n_kv_heads
    # routes of the sampled heads: a sparse candidate per head in turn (the oracle's own probe builds the indices)
    sparse = [c for c in cands if c.pattern != PT.DENSE]
    sets, names = {}, []
    for t, h in enumerate(heads):
        Qf, Kf = bf16_bits_to_f64(Lq["Q"][h]), bf16_bits_to_f64(L["K"][h // G])
        pr = OP.probe_rows(Qf, Kf, spec.n)
        cand = sparse[(t * 5 + 1) % len(sparse)]
        names.append(f"head {h}: pattern {cand.pattern} ({cand.b0},{cand.b1})")
        bs = OP.block_scores(Qf, Kf, 0, spec.n) if cand.pattern == PT.BLOCK_SPARSE else None
        sets[h] = PT.build_indices(cand, 0, spec.n, pr.vert, pr.slash, bs)
    Lfull = {"Q": [Lq["Q"].get(h) for h in range(spec.n_q_heads)], "K": L["K"], "V": L["V"]}
    vals, times = [], []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        tf, desc, cores, _ = oracle_sample(Lfull, spec, cands, None, lambda h: sets[h], None,
                                           budget_s=max(2.0, 60.0 / max(1, args.steps + args.warmup)), n_heads=4,
                                           routes="with one fixed sparse candidate per sampled head, index lists from the "
                                                  "oracle's own probe (no GPU routes: " + "; ".join(names) + ")")
        if it >= args.warmup:
            vals.append(tf); times.append((time.perf_counter() - t0) * 1e3)
    v = float(np.mean(vals))
    out = {"impl": "reference", "metric": metric, "value": v, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": float(np.mean(times)), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
           "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": desc},
           "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
