"""Call sequence of one routed prefill attention layer (the six-step procedure of Section 3.4).

This is the public, user-level entry of the package: it owns the device buffers of one layer and enqueues the
C-ABI calls in order on the current CUDA stream.  It contains no arithmetic of the method: every step runs in the
library's kernels or host functions (profile_costs only times launches and hands the times to the library).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

from . import binding as rs


def default_library() -> List[tuple]:
    """13-candidate online library: four budgets per sparse family by increasing budget, then dense."""
    lib = [(rs.RS_A_SHAPE, 128, w) for w in (1024, 2048, 4096, 8192)]
    lib += [(rs.RS_VERTICAL_SLASH, kv, ks) for kv, ks in ((500, 3048), (1000, 6096), (2000, 12192), (4000, 24384))]
    lib += [(rs.RS_BLOCK_SPARSE, kb, 0) for kb in (50, 100, 200, 400)]
    lib += [(rs.RS_DENSE, 0, 0)]
    return lib


def dense_flops(seg_bounds: Sequence[int], n_q_heads: int, d: int = 128) -> int:
    n = seg_bounds[-1]
    return 4 * d * n_q_heads * (n * (n + 1) // 2)


def probe_flops(seg_bounds: Sequence[int], n_q_heads: int, d: int = 128) -> int:
    tot = 0
    for q0, q1 in zip(seg_bounds[:-1], seg_bounds[1:]):
        tot += 2 * 64 * q1 * d * n_q_heads + 2 * d * n_q_heads * ((q1 // 64) * (q1 // 64 + 1) // 2 - (q0 // 64) * (q0 // 64 + 1) // 2)
    return tot


@dataclass
class RouteConfig:
    budget_frac: float = 0.15          # layer budget T as a fraction of the dense FLOPs of the layer
    alpha: float = 1.0
    delta_q: float = 0.0
    cert_max: Optional[float] = 0.05   # None disables the fallback step
    cert_mode: int = rs.RS_CERT_REL
    expand_first: bool = True
    rescue_any: bool = False           # before dense, the cheapest sparse candidate of any family that passes
    beta: float = 0.0                  # weight of the calibrated predictor e of Eq. 4 (needs use_calibration())
    backfill: bool = False             # spend leftover budget on the best risk decrease per added cost
    mixture_u: bool = False            # u of Eq. 4 from the recent / uniform / boundary rows of the query mixture
    global_pattern: bool = False       # comparison router: one candidate for the whole layer (Section 4, baselines)
    mixture_lists: bool = False        # vertical / slash lists ranked by the query mixture of Eq. 3 (four 16-row runs:
                                       # boundary, two uniformly spaced, recent) instead of the last 64 rows alone


class _IdxView:
    """An rs_index_set struct that points into arrays owned by IndexSet objects."""

    def __init__(self, c_struct):
        self.c = c_struct


class RoutedPrefillLayer:
    """Device buffers and call order for one layer; reuse one instance for every layer of the same shape."""

    def __init__(self, problem: rs.Problem, library: Optional[Sequence[Sequence[int]]] = None,
                 route: Optional[RouteConfig] = None, out_dtype=torch.bfloat16, device="cuda"):
        self.p = problem
        self.cands = list(library) if library is not None else default_library()
        self.lib = rs.make_library(self.cands)
        self.cfg = route or RouteConfig()
        p, S, Hq, Hkv, n = problem, problem.n_segments, problem.n_q_heads, problem.n_kv_heads, problem.n_keys
        f32 = dict(dtype=torch.float32, device=device)
        self.vert = torch.empty((S, Hq, 4, n), **f32)
        self.slash = torch.empty((S, Hq, 4, n), **f32)
        self.lse_probe = torch.empty((Hq, S, 64), **f32)
        self.qpool = torch.empty((Hq, n // 64, 128), **f32)
        self.kpool = torch.empty((Hkv, n // 64, 128), **f32)
        self.vmax = torch.empty((S, Hkv), **f32)
        self.stats = torch.zeros((p.n_items, len(self.cands), 5), dtype=torch.int64, device=device)
        self.idx_eval = rs.IndexSet.for_library(p, self.lib, materialised=False, device=device)
        self.idx = rs.IndexSet.for_library(p, self.lib, materialised=True, device=device)
        # online routing reuses the evaluation's vertical-slash lists: materialise only block-sparse rows, and hand the
        # attention call the evaluation's vertical-slash arrays next to the materialised block-sparse arrays
        e, m = self.idx_eval.c, self.idx.c
        self._idx_bs_only = rs.rs_index_set(0, m.kv_cap, m.ks_cap, m.nd_cap, m.bs_rows, m.kb_cap, m.vs_cols, m.vs_offs,
                                            m.vs_diag, m.vs_count, m.bs_blk, m.bs_count)
        self._idx_hybrid = rs.rs_index_set(e.n_vs_slots, e.kv_cap, e.ks_cap, e.nd_cap, m.bs_rows, m.kb_cap, e.vs_cols,
                                           e.vs_offs, e.vs_diag, e.vs_count, m.bs_blk, m.bs_count)
        self._reuse_eval = False
        self.choice = torch.zeros(p.n_items, dtype=torch.int32, device=device)
        self.report = torch.zeros(24, dtype=torch.uint8, device=device)
        self.O = torch.empty((Hq, n, 128), dtype=out_dtype, device=device)
        self.lse_sel = torch.empty((Hq, n), **f32)
        self.onorm = torch.empty((Hq, n), **f32)
        self.counters = torch.zeros(2, dtype=torch.int64, device=device)
        self.status = rs.new_status(device)
        self.ws = rs.new_workspace(p, self.lib, device)
        rows = []
        for s in range(S):
            rows += list(range(p.seg_bounds[s + 1] - 64, p.seg_bounds[s + 1]))
        self.probe_rows = torch.tensor(rows, dtype=torch.int32, device=device)
        R = len(rows)
        self.m_row = torch.empty((Hq, R), **f32)
        self.cert_row = torch.empty((Hq, R), **f32)
        self.m_head = torch.empty((Hq,), **f32)
        self.cert_head = torch.empty((Hq, 2), **f32)
        self.prm = rs.rs_route_params()
        self.one_call = True        # forward() = one rs_routed_prefill_layer call where that entry point covers the pass
        self._bufs = None
        self._forced = None
        self.events = None
        self.covmix = torch.zeros((p.n_items, len(self.cands), 4), dtype=torch.int64, device=device)
        self.regressor = None       # dict(w, bp_z, bp_e, g) from calibrate(); used when cfg.beta > 0
        self.e_risk = torch.zeros((p.n_items, len(self.cands)), dtype=torch.float64, device=device)
        self.cost_table = None      # int64 [n_items, n_cand] measured kernel time (ns); None: FLOPs of the selected pairs
        self.cost_budget = None     # layer budget in the table's unit
        self.cost_t_probe = 0

    def _layer_buffers(self):
        if self._bufs is None:
            b = rs.rs_layer_buffers()
            for name in ("vert", "slash", "lse_probe", "qpool", "kpool", "vmax", "stats", "choice", "report", "O",
                         "lse_sel", "onorm", "counters", "probe_rows", "m_row", "cert_row", "m_head", "cert_head"):
                setattr(b, name, getattr(self, name).data_ptr())
            b.descr = None
            b.idx_eval, b.idx = self.idx_eval.c, self.idx.c
            b.o_dtype = 1 if self.O.dtype == torch.float32 else 0
            b.n_probe_rows = int(self.probe_rows.numel())
            self._bufs = b
        self._bufs.O = self.O.data_ptr()          # StreamedPrefill rotates the output buffer between passes
        return self._bufs

    # ------------------------------------------------------------------ steps (each only enqueues kernels)
    def probe(self, Q, K, V, lazy_qpool: bool = False):
        """lazy_qpool: pool only the Q rows candidate evaluation reads; pool_routed_queries() adds the rest for the
        heads that end up routed to block-sparse (reading all of Q is the largest stream of the probe)."""
        rs.rs_probe(self.p, Q, K, V, self.vert, self.slash, self.lse_probe, self.qpool, self.kpool, self.vmax, None,
                    self.ws, self.status, flags=rs.RS_PROBE_QPOOL_LAST_ONLY if lazy_qpool else 0)

    def pool_routed_queries(self, Q):
        rs.rs_pool_queries(self.p, Q, self.lib, self.choice, self.qpool, self.status)

    def mixture_probe(self, Q, K):
        """Column and diagonal masses of the query mixture at key resolution (rs_probe_runs) into buffers of their own;
        the run starts come from the library (rs_mixture_runs)."""
        if getattr(self, "_mix", None) is None:
            f32 = dict(dtype=torch.float32, device=self.O.device)
            p = self.p
            self._mix = dict(vert=torch.empty_like(self.vert), slash=torch.empty_like(self.slash),
                             lse=torch.empty((p.n_q_heads, p.n_segments, 64), **f32),
                             runs=[rs.rs_mixture_runs(p.seg_bounds[s], p.seg_bounds[s + 1]) for s in range(p.n_segments)])
        m = self._mix
        rs.rs_probe_runs(self.p, Q, K, m["runs"], m["vert"], m["slash"], m["lse"], self.ws, self.status)

    def evaluate_candidates(self):
        if self.cfg.mixture_lists and getattr(self, "_mix", None) is not None:
            m = self._mix
            rs.rs_build_indices_ranked(self.p, self.lib, self.vert, self.slash, m["vert"], m["slash"], self.qpool,
                                       self.kpool, None, None, self.idx_eval, self.stats, self.ws, self.status)
            return
        rs.rs_build_indices(self.p, self.lib, self.vert, self.slash, self.qpool, self.kpool, None, None,
                            self.idx_eval, self.stats, self.ws, self.status)

    def _fill_route_params(self, forced_dense: Optional[torch.Tensor] = None):
        c, prm = self.cfg, self.prm
        if self.cost_table is not None:
            prm.budget, prm.t_probe = int(self.cost_budget), int(self.cost_t_probe)
        else:
            prm.budget = int(c.budget_frac * dense_flops(self.p.seg_bounds, self.p.n_q_heads))
            prm.t_probe = probe_flops(self.p.seg_bounds, self.p.n_q_heads)
        prm.alpha, prm.delta_q = c.alpha, c.delta_q
        prm.use_cert = 0 if c.cert_max is None else 1
        prm.cert_max = 0.0 if c.cert_max is None else c.cert_max
        prm.cert_mode, prm.expand_first = c.cert_mode, int(c.expand_first)
        prm.rescue_any = int(c.rescue_any)
        prm.backfill = int(c.backfill)
        prm.global_pattern = int(c.global_pattern)
        if c.mixture_u and getattr(self, "_pp_key", None) is not None:
            prm.cov_mix = self.covmix.data_ptr()
            sub = self.pp["sub"]
            for b in range(4):
                prm.mix_rows[b] = (sub[b + 1] - sub[b]) if b + 1 < len(sub) else 0
        else:
            prm.cov_mix = None
        use_e = self.regressor is not None and c.beta > 0.0
        prm.e = self.e_risk.data_ptr() if use_e else None
        prm.beta = float(c.beta) if use_e else 0.0
        self._forced = forced_dense
        prm.forced_dense = None if forced_dense is None else forced_dense.data_ptr()
        prm.fixed_choice = None
        return prm

    def route(self, forced_dense: Optional[torch.Tensor] = None):
        prm = self._fill_route_params(forced_dense)
        rs.rs_route(self.p, self.lib, self.stats, self.cost_table, self.vmax, prm, self.choice, self.report, self.status)

    def materialise(self, reuse_evaluation: bool = False):
        self._reuse_eval = reuse_evaluation and len(self.cands) > 1
        out = _IdxView(self._idx_bs_only) if self._reuse_eval else self.idx
        rs.rs_build_indices(self.p, self.lib, self.vert, self.slash, self.qpool, self.kpool, None, self.choice,
                            out, None, self.ws, self.status)

    def attention(self, Q, K, V):
        idx = _IdxView(self._idx_hybrid) if self._reuse_eval else self.idx
        rs.rs_sparse_prefill_attn(self.p, Q, K, V, self.lib, idx, self.choice, self.O, self.lse_sel, self.onorm,
                                  self.counters, self.ws, self.status)

    def attention_split(self, Q, K, V, heads_per_launch: int):
        """The same attention work as attention(), issued as one launch per group of `heads_per_launch` consecutive
        query heads (a KV group, or a single head) instead of one launch for all heads: the launch-fragmentation
        ablation of Section 3.4 / Table 3.  Single-segment problems only; every launch is the ordinary
        rs_sparse_prefill_attn call on slices of the layer's tensors and index arrays."""
        p = self.p
        assert p.n_segments == 1, "attention_split covers single-segment problems"
        Hq, Hkv, n = p.n_q_heads, p.n_kv_heads, p.n_keys
        group = Hq // Hkv
        assert heads_per_launch in (1, group) or heads_per_launch % group == 0
        nb, n_cand = n // 64, len(self.cands)
        full = self._idx_hybrid if self._reuse_eval else self.idx.c
        eval_layout = self._reuse_eval
        if not hasattr(self, "_sub_problems"):
            self._sub_problems = {}
        for h0 in range(0, Hq, heads_per_launch):
            hn = heads_per_launch
            kv0, kvn = h0 // group, max(1, hn // group)
            key = (hn, kvn)
            if key not in self._sub_problems:
                self._sub_problems[key] = rs.Problem(hn, kvn, n)
            sp = self._sub_problems[key]
            slot0 = h0 * n_cand if eval_layout else h0           # first vertical-slash slot of the slice
            n_slots = hn * n_cand if eval_layout else hn
            sub = rs.rs_index_set(n_slots, full.kv_cap, full.ks_cap, full.nd_cap, hn * nb, full.kb_cap,
                                  full.vs_cols + 4 * slot0 * full.kv_cap, full.vs_offs + 4 * slot0 * full.ks_cap,
                                  full.vs_diag + 4 * slot0 * full.nd_cap, full.vs_count + 16 * slot0,
                                  full.bs_blk + 4 * h0 * nb * full.kb_cap, full.bs_count + 4 * h0 * nb)
            rs.rs_sparse_prefill_attn(sp, Q[h0:h0 + hn], K[kv0:kv0 + kvn], V[kv0:kv0 + kvn], self.lib, _IdxView(sub),
                                      self.choice[h0:h0 + hn], self.O[h0:h0 + hn], self.lse_sel[h0:h0 + hn],
                                      self.onorm[h0:h0 + hn], self.counters, self.ws, self.status)

    def certificate(self):
        p = self.p
        rs.rs_certificate(p.n_q_heads, p.n_kv_heads, p.n_keys, self.lse_sel, self.lse_probe, self.probe_rows,
                          self.vmax[p.n_segments - 1], self.onorm, self.cfg.delta_q, self.m_row, self.cert_row, None,
                          self.m_head, self.cert_head, self.status)

    # ------------------------------------------------------------------ Eq. 3 in its general form + descriptors
    def pooled_probe(self, Q, K, g: int = 64, mixture=(32, 16, 16)):
        """Mixture-of-rows probe against keys pooled over width g (Eq. 3) and the three descriptors of Section 3.2.
        Returns the descriptor tensor [n_seg][Hq][4] (entropy, local-band mass, agreement between the recent and the
        uniform rows, mean number of visible blocks); probabilities and block masses stay in self.pp."""
        p = self.p
        key = (g, tuple(mixture))
        if getattr(self, "_pp_key", None) != key:
            dev = self.O.device
            r = sum(mixture)
            f32 = dict(dtype=torch.float32, device=dev)
            rows = [rs.mixture_rows(p.seg_bounds[s], p.seg_bounds[s + 1], *mixture) for s in range(p.n_segments)]
            nbg = p.n_keys // g
            self.pp = dict(rows=torch.tensor(rows, dtype=torch.int32, device=dev),
                           sub=[0, mixture[0], mixture[0] + mixture[1], r],
                           A=torch.empty((p.n_segments, p.n_q_heads, r, nbg), **f32),
                           lse=torch.empty((p.n_segments, p.n_q_heads, r), **f32),
                           col=torch.empty((p.n_segments, p.n_q_heads, 3, nbg), **f32),
                           diag=torch.empty((p.n_segments, p.n_q_heads, 3, nbg), **f32),
                           descr=torch.empty((p.n_segments, p.n_q_heads, 4), **f32),
                           scratch=torch.empty(rs.rs_probe_pooled_scratch_floats(p, r), **f32))
            self._pp_key = key
        pp = self.pp
        rs.rs_probe_pooled(p, Q, K, pp["rows"], g, pp["sub"], pp["A"], pp["lse"], pp["col"], pp["diag"], pp["descr"],
                           pp["scratch"], self.status)
        return pp["descr"]

    # ------------------------------------------------------------------ offline calibration (Section 3.5)
    def profile_costs(self, Q, K, V, reps: int = 3):
        """Hardware profiling of the pattern library (Section 3.1, 3.5): every candidate runs as the route of all
        heads and its attention launch is timed (median of `reps`, CUDA events).  The measured time of a candidate is
        (the maximum is reported as its tail latency) is split over the items in proportion to their pair counts and stored as the int64 nanosecond cost table the
        router reads; the layer budget becomes budget_frac x the dense candidate's measured time and t_probe the
        measured probe + evaluation time.  Synchronises; meant to run once per (library, length), outside the hot path."""
        import numpy as np
        p, n_cand = self.p, len(self.cands)
        ev = lambda: torch.cuda.Event(enable_timing=True)
        self.probe(Q, K, V)
        self.evaluate_candidates()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record(); self.probe(Q, K, V); self.evaluate_candidates(); b.record()
        torch.cuda.synchronize()
        t_probe_ns = a.elapsed_time(b) * 1e6
        ms, tail = np.zeros(n_cand), np.zeros(n_cand)     # median and tail (maximum of the repetitions)
        saved = self.choice.clone()
        for c in range(n_cand):
            self.choice.fill_(c)
            self.materialise(reuse_evaluation=True)
            self.attention(Q, K, V)
            ts = []
            for _ in range(reps):
                a, b = ev(), ev()
                a.record(); self.attention(Q, K, V); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            ms[c] = float(np.median(ts))
            tail[c] = float(np.max(ts))
        self.choice.copy_(saved)
        table = rs.rs_cost_table_from_times(ms, self.stats.cpu().numpy()[:, :, 4].astype(np.uint64))
        dense_c = [i for i, c in enumerate(self.cands) if c[0] == rs.RS_DENSE][0]
        self.cost_table = torch.from_numpy(table).to(self.O.device)
        self.cost_budget = int(self.cfg.budget_frac * ms[dense_c] * 1e6)
        self.cost_t_probe = int(t_probe_ns)
        return {"candidate_ms": ms.tolist(), "candidate_ms_tail": tail.tolist(), "t_probe_ms": t_probe_ns * 1e-6,
                "budget_ms": self.cost_budget * 1e-6}

    def use_flop_costs(self):
        self.cost_table = None

    def use_calibration(self, calib: dict, beta: Optional[float] = None):
        """Installs the result of calibrate(): the one-sided residual quantile delta_q and the predictor e of Eq. 4."""
        self.cfg.delta_q = float(calib["delta_q"])
        self.regressor = dict(calib["regressor"])
        if beta is not None:
            self.cfg.beta = float(beta)

    def mixture_coverage(self, Q, K):
        """Coverage of every candidate on the rows of the query mixture (pooled probe at g = 64), the input of the
        subset-disagreement u of Eq. 4; needs evaluate_candidates()."""
        self.pooled_probe(Q, K, g=64)
        pp = self.pp
        rs.rs_mixture_coverage(self.p, self.lib, pp["A"], pp["rows"], pp["sub"], self.idx_eval, self.qpool, self.kpool,
                               self.covmix, self.status)
        return self.covmix

    def predict_error(self, Q, K):
        """Descriptors (pooled mixture probe) and the predictor e for every (item, candidate); needs evaluate_candidates()."""
        r = self.regressor
        descr = self.pooled_probe(Q, K, g=int(r["g"]))
        rs.rs_regressor_eval(self.p, self.lib, self.stats, descr, r["w"], r["bp_z"], r["bp_e"], self.e_risk, self.status)
        return self.e_risk

    # ------------------------------------------------------------------ whole layer
    def forward(self, Q, K, V, fixed_choice: Optional[torch.Tensor] = None,
                forced_dense: Optional[torch.Tensor] = None, record_events: bool = False) -> torch.Tensor:
        """Routed sparse prefill attention of one layer; returns O (device). Nothing synchronises."""
        staged = (record_events or self.cfg.mixture_u or self.cfg.mixture_lists
                  or (self.regressor is not None and self.cfg.beta > 0.0) or not self.one_call)
        if not staged:
            # the whole pass as one library call; the staged path below issues the same calls one by one (needed for
            # per-stage timing and for the steps the one-call entry point does not cover: mixture coverage, predictor e)
            prm = self._fill_route_params(forced_dense if fixed_choice is None else None)
            prm.fixed_choice = None if fixed_choice is None else fixed_choice.data_ptr()
            rs.rs_routed_prefill_layer(self.p, Q, K, V, self.lib, prm, self.cost_table, self._layer_buffers(), self.ws,
                                       self.status)
            prm.fixed_choice = None
            self._reuse_eval = fixed_choice is None and len(self.cands) > 1
            self.events = None
            return self.O
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(7)] if record_events else None
        mark = (lambda i: ev[i].record()) if record_events else (lambda i: None)
        mark(0)
        lazy = not self.cfg.mixture_u        # the mixture coverage reads pooled queries of blocks all over the segment
        self.probe(Q, K, V, lazy_qpool=lazy)
        if self.cfg.mixture_lists and fixed_choice is None:
            self.mixture_probe(Q, K)
        mark(1)
        if fixed_choice is None:
            self.evaluate_candidates()
            if self.cfg.mixture_u:
                self.mixture_coverage(Q, K)
            if self.regressor is not None and self.cfg.beta > 0.0:
                self.predict_error(Q, K)
            mark(2)
            self.route(forced_dense)
        else:
            self.choice.copy_(fixed_choice)
            mark(2)
        mark(3)
        if lazy:
            self.pool_routed_queries(Q)
        self.materialise(reuse_evaluation=fixed_choice is None)
        mark(4)
        self.attention(Q, K, V)
        mark(5)
        self.certificate()
        mark(6)
        self.events = ev
        return self.O

    def forward_from_hidden(self, X, W, rope_cos, rope_sin, forced_dense: Optional[torch.Tensor] = None,
                            record_events: bool = False) -> torch.Tensor:
        """The layer pass with its producer in front (Section 3.4: the probe as a reduction fused with the projection
        kernels): rs_qkv_rope_project writes Q, K, V into buffers owned by the layer together with the pooled queries
        and keys and the block maxima of the value norms, so rs_probe runs only its two passes over K (no pooling, no
        stream over V) and no query pooling follows the routing.  X [n, d_model] bf16, W [(Hq + 2 Hkv) * 128, d_model]
        bf16, rope tables fp32 [n, 64].  Events (record_events): projection, probe, evaluate, route, materialise,
        attention, certificate."""
        p = self.p
        if getattr(self, "_qkv", None) is None:
            bf = dict(dtype=torch.bfloat16, device=self.O.device)
            self._qkv = (torch.empty((p.n_q_heads, p.n_keys, 128), **bf), torch.empty((p.n_kv_heads, p.n_keys, 128), **bf),
                         torch.empty((p.n_kv_heads, p.n_keys, 128), **bf))
            self._vbmax = torch.empty((p.n_kv_heads, p.n_keys // 64), dtype=torch.float32, device=self.O.device)
        Q, K, V = self._qkv
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(8)] if record_events else None
        mark = (lambda i: ev[i].record()) if record_events else (lambda i: None)
        mark(0)
        rs.rs_qkv_rope_project(X, W, rope_cos, rope_sin, p.n_q_heads, p.n_kv_heads, Q, K, V, self.qpool, self.kpool,
                               self._vbmax, self.status)
        mark(1)
        rs.rs_probe(p, Q, K, V, self.vert, self.slash, self.lse_probe, None, None, None, None, self.ws, self.status)
        rs.rs_value_norm_max(p, self._vbmax, self.vmax, self.status)
        mark(2)
        self.evaluate_candidates()
        mark(3)
        self.route(forced_dense)
        mark(4)
        self.materialise(reuse_evaluation=True)
        mark(5)
        self.attention(Q, K, V)
        mark(6)
        self.certificate()
        mark(7)
        self.events_hidden = ev
        return self.O

    def stage_ms(self):
        """Milliseconds per stage of the last forward(record_events=True): probe, evaluate, route, materialise,
        attention, certificate (synchronises)."""
        torch.cuda.synchronize()
        e = self.events
        names = ["probe", "evaluate", "route", "materialise", "attention", "certificate"]
        return {names[i]: e[i].elapsed_time(e[i + 1]) for i in range(6)}

    def download_index_lists(self, choice):
        """The routed candidates' index lists as host arrays, one dict per item (synchronises): vertical-slash items
        carry V (columns), S (offsets), D (block diagonals); block-sparse items carry blk, one array of key blocks per
        query block of the segment.  Knows where the lists sit (the evaluation's slots when they were reused)."""
        p = self.p
        nb, n_cand = p.n_keys // 64, len(self.cands)
        vs = self.idx_eval if self._reuse_eval else self.idx
        cnt = vs.vs_count.cpu().numpy()
        cols, offs, diag = (t.cpu().numpy() for t in (vs.vs_cols, vs.vs_offs, vs.vs_diag))
        blk, bcnt = self.idx.bs_blk.cpu().numpy(), self.idx.bs_count.cpu().numpy()
        out = []
        for item in range(p.n_items):
            s, h = divmod(item, p.n_q_heads)
            c = int(choice[item])
            d = dict(pattern=self.cands[c][0], q0=p.seg_bounds[s], q1=p.seg_bounds[s + 1])
            if d["pattern"] == rs.RS_VERTICAL_SLASH:
                sl = item * n_cand + c if self._reuse_eval else item
                d.update(V=cols[sl, :cnt[sl, 0]], S=offs[sl, :cnt[sl, 1]], D=diag[sl, :cnt[sl, 2]])
            elif d["pattern"] == rs.RS_BLOCK_SPARSE:
                d["blk"] = [blk[h * nb + qb, :bcnt[h * nb + qb]] for qb in range(d["q0"] // 64, d["q1"] // 64)]
            out.append(d)
        return out

    def route_report(self):
        import numpy as np
        r = self.report.cpu().numpy()
        return dict(total_cost=int(r[:8].view(np.int64)[0]), total_risk=float(r[8:16].view(np.float64)[0]),
                    n_fallback=int(r[16:20].view(np.int32)[0]), feasible=int(r[20:24].view(np.int32)[0]))


def prefill_from_host(layer: RoutedPrefillLayer, Q_host: torch.Tensor, K_host: torch.Tensor, V_host: torch.Tensor,
                      O_host: torch.Tensor, dev_bufs=None) -> torch.Tensor:
    """End-to-end call with pinned HOST buffers: copies Q, K, V to the device, runs the layer, copies O back."""
    if dev_bufs is None:
        dev_bufs = tuple(torch.empty_like(t, device=layer.O.device) for t in (Q_host, K_host, V_host))
    Qd, Kd, Vd = dev_bufs
    Qd.copy_(Q_host, non_blocking=True)
    Kd.copy_(K_host, non_blocking=True)
    Vd.copy_(V_host, non_blocking=True)
    O = layer.forward(Qd, Kd, Vd)
    O_host.copy_(O, non_blocking=True)
    return O_host


class GraphedPrefill:
    """A layer pass captured once into a CUDA graph and replayed: for launch-bound sizes (a 4K layer takes 0.26 ms issued
    call by call and 0.13 ms replayed).  The graph reads the Q, K, V buffers it was captured with, so run() copies new
    inputs into those buffers (device to device) unless it is handed the very same tensors; the routes are recomputed on
    the device at every replay.  The first, eager pass also does the one-time per-device kernel set-up, which must stay
    outside the capture."""

    def __init__(self, layer: RoutedPrefillLayer, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, **forward_kw):
        self.layer, self.Q, self.K, self.V = layer, Q, K, V
        layer.forward(Q, K, V, **forward_kw)
        torch.cuda.synchronize()
        rs.check_status(layer.status, "eager pass before the capture")
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            layer.forward(Q, K, V, **forward_kw)

    def run(self, Q: Optional[torch.Tensor] = None, K: Optional[torch.Tensor] = None,
            V: Optional[torch.Tensor] = None) -> torch.Tensor:
        for dst, src in ((self.Q, Q), (self.K, K), (self.V, V)):
            if src is not None and src.data_ptr() != dst.data_ptr():
                dst.copy_(src, non_blocking=True)
        self.graph.replay()
        return self.layer.O


class StreamedPrefill:
    """Layer passes fed from pinned HOST buffers with the copies overlapped with the kernels: three streams (host to
    device, compute, device to host) and two device buffer sets, so that while pass k computes, the inputs of pass k + 1
    arrive and the output of pass k - 1 leaves.  Every pass still copies its own Q, K, V in and its own O out; only the
    order on the copy engines and the SMs is pipelined.  submit() enqueues one pass and returns immediately; finish()
    makes the caller's current stream wait for everything submitted."""

    def __init__(self, layer: RoutedPrefillLayer, n_buffers: int = 2):
        self.layer = layer
        dev = layer.O.device
        p = layer.p
        shape_q = (p.n_q_heads, p.n_keys, 128)
        shape_kv = (p.n_kv_heads, p.n_keys, 128)
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.n = n_buffers
        self.Q = [torch.empty(shape_q, **bf) for _ in range(n_buffers)]
        self.K = [torch.empty(shape_kv, **bf) for _ in range(n_buffers)]
        self.V = [torch.empty(shape_kv, **bf) for _ in range(n_buffers)]
        self.O = [layer.O] + [torch.empty_like(layer.O) for _ in range(n_buffers - 1)]
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
        ev = lambda: [torch.cuda.Event() for _ in range(n_buffers)]
        self.in_done, self.run_done, self.out_done = ev(), ev(), ev()
        self.k = 0

    def submit(self, Q_host, K_host, V_host, O_host, **forward_kw):
        b = self.k % self.n
        first_use = self.k < self.n
        cur = torch.cuda.current_stream()
        with torch.cuda.stream(self.s_in):
            self.s_in.wait_stream(cur) if self.k == 0 else None
            if not first_use:
                self.s_in.wait_event(self.run_done[b])          # the pass that last read this input set is done
            self.Q[b].copy_(Q_host, non_blocking=True)
            self.K[b].copy_(K_host, non_blocking=True)
            self.V[b].copy_(V_host, non_blocking=True)
            self.in_done[b].record(self.s_in)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(self.in_done[b])
            if not first_use:
                self.s_run.wait_event(self.out_done[b])         # the output buffer has been copied out
            self.layer.O = self.O[b]
            self.layer.forward(self.Q[b], self.K[b], self.V[b], **forward_kw)
            self.run_done[b].record(self.s_run)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.run_done[b])
            O_host.copy_(self.O[b], non_blocking=True)
            self.out_done[b].record(self.s_out)
        self.k += 1

    def finish(self):
        cur = torch.cuda.current_stream()
        for s in (self.s_in, self.s_run, self.s_out):
            cur.wait_stream(s)
        self.layer.O = self.O[0]
