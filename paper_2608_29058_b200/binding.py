"""ctypes binding of the C ABI in include/routesparse.h -- argument marshalling only.

Every function has the name and argument order of its C counterpart; tensors are torch CUDA tensors whose
data pointers are passed through.  Nothing is computed here: if the shared library is missing the import of
the first entry point fails loudly (there is no fallback path).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

RS_DENSE, RS_A_SHAPE, RS_VERTICAL_SLASH, RS_BLOCK_SPARSE = 0, 1, 2, 3
RS_CERT_ABS, RS_CERT_REL = 0, 1
RS_STATUS_WORDS = 8
RS_OK = 0

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "librs_b200.so")
_lib = None


class rs_candidate(C.Structure):
    _fields_ = [("pattern", C.c_int32), ("b0", C.c_int32), ("b1", C.c_int32), ("flags", C.c_int32)]


class rs_problem(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("n_keys", C.c_int32), ("n_segments", C.c_int32), ("seg_bounds", C.POINTER(C.c_int32))]


class rs_index_set(C.Structure):
    _fields_ = [("n_vs_slots", C.c_int32), ("kv_cap", C.c_int32), ("ks_cap", C.c_int32), ("nd_cap", C.c_int32),
                ("bs_rows", C.c_int32), ("kb_cap", C.c_int32),
                ("vs_cols", C.c_void_p), ("vs_offs", C.c_void_p), ("vs_diag", C.c_void_p), ("vs_count", C.c_void_p),
                ("bs_blk", C.c_void_p), ("bs_count", C.c_void_p)]


class rs_route_params(C.Structure):
    _fields_ = [("budget", C.c_int64), ("t_probe", C.c_int64), ("alpha", C.c_double), ("delta_q", C.c_double),
                ("cert_max", C.c_double), ("use_cert", C.c_int32), ("cert_mode", C.c_int32),
                ("expand_first", C.c_int32), ("rescue_any", C.c_int32),
                ("forced_dense", C.c_void_p), ("fixed_choice", C.c_void_p), ("e", C.c_void_p), ("beta", C.c_double),
                ("backfill", C.c_int32), ("global_pattern", C.c_int32), ("cov_mix", C.c_void_p), ("mix_rows", C.c_int32 * 4)]


class rs_layer_buffers(C.Structure):
    _fields_ = [("vert", C.c_void_p), ("slash", C.c_void_p), ("lse_probe", C.c_void_p), ("qpool", C.c_void_p),
                ("kpool", C.c_void_p), ("vmax", C.c_void_p), ("descr", C.c_void_p), ("stats", C.c_void_p),
                ("idx_eval", rs_index_set), ("idx", rs_index_set), ("choice", C.c_void_p), ("report", C.c_void_p),
                ("O", C.c_void_p), ("o_dtype", C.c_int32), ("n_probe_rows", C.c_int32), ("lse_sel", C.c_void_p),
                ("onorm", C.c_void_p), ("counters", C.c_void_p), ("probe_rows", C.c_void_p), ("m_row", C.c_void_p),
                ("cert_row", C.c_void_p), ("m_head", C.c_void_p), ("cert_head", C.c_void_p)]


EXPORTS = ["rs_error_string", "rs_version", "rs_workspace_bytes", "rs_probe", "rs_build_indices", "rs_route",
           "rs_sparse_prefill_attn", "rs_dense_prefill_attn", "rs_dense_prefill_attn_noalloc", "rs_certificate",
           "rs_selftest_wait_timeout", "rs_probe_pooled", "rs_probe_pooled_scratch_floats", "rs_regressor_eval",
           "rs_output_error", "rs_mixture_coverage", "rs_pool_queries", "rs_routed_prefill_layer",
           "rs_qkv_rope_project", "rs_value_norm_max", "rs_probe_runs", "rs_build_indices_ranked",
           "rs_mixture_rows", "rs_mixture_runs", "rs_calibration_fit", "rs_cost_table_from_times"]


def lib_path() -> str:
    return _LIB_PATH


def load() -> C.CDLL:
    """Loads the shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2608_29058_b200.build` "
                               "(or __graft_entry__.build()); this package has no CPU or eager fallback")
        _lib = C.CDLL(_LIB_PATH)
        _lib.rs_error_string.restype = C.c_char_p
        _lib.rs_error_string.argtypes = [C.c_int]
        for name in EXPORTS[1:]:
            getattr(_lib, name).restype = C.c_int
    return _lib


class RouteSparseError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != RS_OK:
        raise RouteSparseError(f"{what} failed: {rc} ({load().rs_error_string(rc).decode()})")


def _ptr(t: Optional[torch.Tensor]) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Problem:
    """Host-side description of one layer: head geometry, length and segment bounds."""
    n_q_heads: int
    n_kv_heads: int
    n_keys: int
    seg_bounds: Sequence[int] = ()
    head_dim: int = 128

    def __post_init__(self):
        sb = list(self.seg_bounds) or [0, self.n_keys]
        self._sb = (C.c_int32 * len(sb))(*sb)
        self.seg_bounds = sb
        self.c = rs_problem(self.n_q_heads, self.n_kv_heads, self.head_dim, self.n_keys, len(sb) - 1,
                            C.cast(self._sb, C.POINTER(C.c_int32)))

    @property
    def n_segments(self) -> int:
        return len(self.seg_bounds) - 1

    @property
    def n_items(self) -> int:
        return self.n_segments * self.n_q_heads


def make_library(cands: Sequence[Sequence[int]]):
    """[(pattern, b0, b1), ...] -> ctypes array of rs_candidate."""
    arr = (rs_candidate * len(cands))()
    for i, c in enumerate(cands):
        c = list(c) + [0] * (4 - len(c))
        arr[i] = rs_candidate(int(c[0]), int(c[1]), int(c[2]), int(c[3]))
    return arr


class IndexSet:
    """Device storage for an rs_index_set (allocation only)."""

    def __init__(self, n_vs_slots: int, kv_cap: int, ks_cap: int, nd_cap: int, bs_rows: int, kb_cap: int,
                 device="cuda"):
        i32 = dict(dtype=torch.int32, device=device)
        self.vs_cols = torch.zeros((max(1, n_vs_slots), max(1, kv_cap)), **i32)
        self.vs_offs = torch.zeros((max(1, n_vs_slots), max(1, ks_cap)), **i32)
        self.vs_diag = torch.zeros((max(1, n_vs_slots), max(1, nd_cap)), **i32)
        self.vs_count = torch.zeros((max(1, n_vs_slots), 4), **i32)
        self.bs_blk = torch.zeros((max(1, bs_rows), max(1, kb_cap)), **i32)
        self.bs_count = torch.zeros((max(1, bs_rows),), **i32)
        self.c = rs_index_set(n_vs_slots, max(1, kv_cap), max(1, ks_cap), max(1, nd_cap), bs_rows, max(1, kb_cap),
                              self.vs_cols.data_ptr(), self.vs_offs.data_ptr(), self.vs_diag.data_ptr(),
                              self.vs_count.data_ptr(), self.bs_blk.data_ptr(), self.bs_count.data_ptr())

    @staticmethod
    def for_library(p: Problem, lib, materialised: bool, device="cuda") -> "IndexSet":
        kv = max([c.b0 for c in lib if c.pattern == RS_VERTICAL_SLASH] + [0])
        ks = max([c.b1 for c in lib if c.pattern == RS_VERTICAL_SLASH] + [0])
        kb = max([c.b0 for c in lib if c.pattern == RS_BLOCK_SPARSE] + [0])
        nb = p.n_keys // 64
        kv, ks, kb = min(kv, p.n_keys), min(ks, p.n_keys), min(kb, nb)
        if materialised:
            return IndexSet(p.n_items, kv, ks, nb, p.n_q_heads * nb, kb, device)
        return IndexSet(p.n_items * len(lib), kv, ks, nb, p.n_items * len(lib), kb, device)


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(RS_STATUS_WORDS, dtype=torch.int32, device=device)


def rs_version() -> int:
    return load().rs_version()


def rs_error_string(code: int) -> str:
    return load().rs_error_string(code).decode()


def rs_workspace_bytes(p: Problem, lib) -> int:
    out = C.c_size_t(0)
    n = 0 if lib is None else len(lib)
    _check(load().rs_workspace_bytes(C.byref(p.c), lib, n, C.byref(out)), "rs_workspace_bytes")
    return int(out.value)


def new_workspace(p: Problem, lib, device="cuda") -> torch.Tensor:
    return torch.empty(max(256, rs_workspace_bytes(p, lib)), dtype=torch.uint8, device=device)


RS_PROBE_QPOOL_LAST_ONLY = 1


def rs_probe(p: Problem, Q, K, V, vert, slash, lse_probe, qpool, kpool, vmax, descr, ws, status, flags: int = 0):
    _check(load().rs_probe(C.byref(p.c), _ptr(Q), _ptr(K), _ptr(V), _ptr(vert), _ptr(slash), _ptr(lse_probe),
                           _ptr(qpool), _ptr(kpool), _ptr(vmax), _ptr(descr), int(flags), _ptr(ws),
                           C.c_size_t(ws.numel()), _ptr(status), _stream()), "rs_probe")


def rs_probe_runs(p: Problem, Q, K, run_starts, vert, slash, lse_probe, ws, status):
    """Probe on four 16-row runs per segment (the query mixture at key resolution); run_starts: [n_seg][4] ints."""
    flat = [int(x) for row in run_starts for x in row]
    arr = (C.c_int32 * len(flat))(*flat)
    _check(load().rs_probe_runs(C.byref(p.c), _ptr(Q), _ptr(K), arr, _ptr(vert), _ptr(slash), _ptr(lse_probe), _ptr(ws),
                                C.c_size_t(ws.numel()), _ptr(status), _stream()), "rs_probe_runs")


def rs_pool_queries(p: Problem, Q, lib, choice, qpool, status):
    """64-row means of Q for the heads routed to block-sparse (choice None: every head)."""
    n = 0 if lib is None else len(lib)
    _check(load().rs_pool_queries(C.byref(p.c), _ptr(Q), lib, n, _ptr(choice), _ptr(qpool), _ptr(status), _stream()),
           "rs_pool_queries")


def rs_build_indices(p: Problem, lib, vert, slash, qpool, kpool, bscore, choice, out: IndexSet, stats, ws, status):
    _check(load().rs_build_indices(C.byref(p.c), lib, len(lib), _ptr(vert), _ptr(slash), _ptr(qpool), _ptr(kpool),
                                   _ptr(bscore), _ptr(choice), C.byref(out.c), _ptr(stats), _ptr(ws),
                                   C.c_size_t(ws.numel()), _ptr(status), _stream()), "rs_build_indices")


def rs_build_indices_ranked(p: Problem, lib, vert, slash, rank_vert, rank_slash, qpool, kpool, bscore, choice,
                            out: IndexSet, stats, ws, status):
    """rs_build_indices with the line lists ranked by rank_vert / rank_slash (masses of the query mixture)."""
    _check(load().rs_build_indices_ranked(C.byref(p.c), lib, len(lib), _ptr(vert), _ptr(slash), _ptr(rank_vert),
                                          _ptr(rank_slash), _ptr(qpool), _ptr(kpool), _ptr(bscore), _ptr(choice),
                                          C.byref(out.c), _ptr(stats), _ptr(ws), C.c_size_t(ws.numel()), _ptr(status),
                                          _stream()), "rs_build_indices_ranked")


def rs_route(p: Problem, lib, stats, cost, vmax, params: rs_route_params, choice, report, status):
    _check(load().rs_route(C.byref(p.c), lib, len(lib), _ptr(stats), _ptr(cost), _ptr(vmax), C.byref(params),
                           _ptr(choice), _ptr(report), _ptr(status), _stream()), "rs_route")


def rs_routed_prefill_layer(p: Problem, Q, K, V, lib, params: rs_route_params, cost, bufs: rs_layer_buffers, ws, status):
    """The whole layer pass in one library call (probe, evaluation, routing, materialisation, attention, certificate)."""
    _check(load().rs_routed_prefill_layer(C.byref(p.c), _ptr(Q), _ptr(K), _ptr(V), lib, len(lib), C.byref(params),
                                          _ptr(cost), C.byref(bufs), _ptr(ws), C.c_size_t(ws.numel()), _ptr(status),
                                          _stream()), "rs_routed_prefill_layer")


def rs_sparse_prefill_attn(p: Problem, Q, K, V, lib, idx: IndexSet, choice, O, lse_sel, onorm, counters, ws, status):
    o_dtype = 1 if O.dtype == torch.float32 else 0
    _check(load().rs_sparse_prefill_attn(C.byref(p.c), _ptr(Q), _ptr(K), _ptr(V), lib, len(lib), C.byref(idx.c),
                                         _ptr(choice), _ptr(O), o_dtype, _ptr(lse_sel), _ptr(onorm), _ptr(counters),
                                         _ptr(ws), C.c_size_t(ws.numel()), _ptr(status), _stream()),
           "rs_sparse_prefill_attn")


def rs_dense_prefill_attn(p: Problem, Q, K, V, O, lse, onorm, counters, ws, status):
    o_dtype = 1 if O.dtype == torch.float32 else 0
    _check(load().rs_dense_prefill_attn(C.byref(p.c), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), o_dtype, _ptr(lse),
                                        _ptr(onorm), _ptr(counters), _ptr(ws), C.c_size_t(ws.numel()), _ptr(status),
                                        _stream()), "rs_dense_prefill_attn")


def rs_dense_prefill_attn_noalloc(p: Problem, Q, K, V, O, lse, onorm, status):
    """Dense causal attention with the library's built-in scratch: no workspace argument, no allocation."""
    o_dtype = 1 if O.dtype == torch.float32 else 0
    _check(load().rs_dense_prefill_attn_noalloc(C.byref(p.c), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), o_dtype, _ptr(lse),
                                                _ptr(onorm), _ptr(status), _stream()), "rs_dense_prefill_attn_noalloc")


def rs_certificate(n_q_heads: int, n_kv_heads: int, n_keys: int, lse_sel, lse_full, rows, vmax, onorm,
                   delta_q: float, m_row, cert_row, cert_tight, m_head, cert_head, status):
    _check(load().rs_certificate(n_q_heads, n_kv_heads, n_keys, _ptr(lse_sel), _ptr(lse_full), _ptr(rows),
                                 int(rows.numel()), _ptr(vmax), _ptr(onorm), C.c_float(delta_q), _ptr(m_row),
                                 _ptr(cert_row), _ptr(cert_tight), _ptr(m_head), _ptr(cert_head), _ptr(status),
                                 _stream()), "rs_certificate")


def rs_probe_pooled_scratch_floats(p: Problem, r: int) -> int:
    out = C.c_size_t(0)
    _check(load().rs_probe_pooled_scratch_floats(C.byref(p.c), int(r), C.byref(out)), "rs_probe_pooled_scratch_floats")
    return int(out.value)


def mixture_rows(q0: int, q1: int, r_recent: int = 32, r_uniform: int = 16, r_boundary: int = 16):
    """Row ids of the probe's query mixture (Section 3.2) for the segment [q0, q1): rs_mixture_rows of the library."""
    r = r_recent + r_uniform + r_boundary
    out = (C.c_int32 * r)()
    rc = load().rs_mixture_rows(int(q0), int(q1), int(r_recent), int(r_uniform), int(r_boundary), out)
    if rc == -2:
        raise ValueError("segment too short for this mixture")
    _check(rc, "rs_mixture_rows")
    return list(out)


def rs_mixture_runs(q0: int, q1: int):
    """First rows of the four 16-row runs of the query mixture at key resolution (rs_mixture_runs of the library)."""
    out = (C.c_int32 * 4)()
    _check(load().rs_mixture_runs(int(q0), int(q1), out), "rs_mixture_runs")
    return list(out)


def rs_probe_pooled(p: Problem, Q, K, rows, g: int, sub_bounds, A, lse, colmass, diagmass, descr, scratch, status):
    """rows: device int32 [n_seg][r]; sub_bounds: host list of n_sub + 1 ints."""
    r = int(rows.shape[-1])
    sb = (C.c_int32 * len(sub_bounds))(*[int(x) for x in sub_bounds])
    _check(load().rs_probe_pooled(C.byref(p.c), _ptr(Q), _ptr(K), _ptr(rows), r, int(g), sb, len(sub_bounds) - 1,
                                  _ptr(A), _ptr(lse), _ptr(colmass), _ptr(diagmass), _ptr(descr), _ptr(scratch),
                                  _ptr(status), _stream()), "rs_probe_pooled")


def rs_mixture_coverage(p: Problem, lib, A, rows, sub_bounds, idx_eval, qpool, kpool, covmix, status):
    """A: pooled-probe probabilities at g = 64; rows: device int32 [n_seg][r]; covmix: device int64/uint64 [items][cands][4]."""
    r = int(rows.shape[-1])
    sb = (C.c_int32 * len(sub_bounds))(*[int(x) for x in sub_bounds])
    _check(load().rs_mixture_coverage(C.byref(p.c), lib, len(lib), _ptr(A), _ptr(rows), r, sb, len(sub_bounds) - 1,
                                      C.byref(idx_eval.c), _ptr(qpool), _ptr(kpool), _ptr(covmix), _ptr(status),
                                      _stream()), "rs_mixture_coverage")


def rs_regressor_eval(p: Problem, lib, stats, descr, w, bp_z, bp_e, e_out, status):
    """w: 6 host floats; bp_z / bp_e: host lists (breakpoints of the step function); e_out: device float64."""
    wd = (C.c_double * 6)(*[float(x) for x in w])
    n_bp = len(bp_z)
    bz = (C.c_double * max(1, n_bp))(*[float(x) for x in bp_z])
    be = (C.c_double * max(1, n_bp))(*[float(x) for x in bp_e])
    _check(load().rs_regressor_eval(C.byref(p.c), lib, len(lib), _ptr(stats), _ptr(descr), wd, bz, be, n_bp,
                                    _ptr(e_out), _ptr(status), _stream()), "rs_regressor_eval")


def rs_output_error(Oa, Ob, err, norm_a, status):
    n_rows = Oa.numel() // 128
    o_dtype = 1 if Oa.dtype == torch.float32 else 0
    _check(load().rs_output_error(C.c_longlong(n_rows), _ptr(Oa), _ptr(Ob), o_dtype, _ptr(err), _ptr(norm_a),
                                  _ptr(status), _stream()), "rs_output_error")


def rs_qkv_rope_project(X, W, rope_cos, rope_sin, n_q_heads: int, n_kv_heads: int, Q, K, V, qpool, kpool, vbmax, status):
    """QKV projection + rotary embedding with the probe's side outputs (pooled Q / K, block maxima of ||v||^2)."""
    n, dm = int(X.shape[0]), int(X.shape[1])
    _check(load().rs_qkv_rope_project(n, dm, n_q_heads, n_kv_heads, _ptr(X), _ptr(W), _ptr(rope_cos), _ptr(rope_sin),
                                      _ptr(Q), _ptr(K), _ptr(V), _ptr(qpool), _ptr(kpool), _ptr(vbmax), _ptr(status),
                                      _stream()), "rs_qkv_rope_project")


def rs_value_norm_max(p: Problem, vbmax, vmax, status):
    _check(load().rs_value_norm_max(C.byref(p.c), _ptr(vbmax), _ptr(vmax), _ptr(status), _stream()), "rs_value_norm_max")


def rs_calibration_fit(features, target, residual, q: float, max_breakpoints: int = 64):
    """Host statistics of the offline calibration (library function): returns (delta_q, w, bp_z, bp_e)."""
    import numpy as np
    X = np.ascontiguousarray(features, dtype=np.float64)
    y = np.ascontiguousarray(target, dtype=np.float64)
    r = np.ascontiguousarray(residual, dtype=np.float64)
    n, nf = X.shape
    dq, nbp = C.c_double(0.0), C.c_int(0)
    w = np.zeros(nf); bz = np.zeros(n); be = np.zeros(n)
    dp = lambda a: a.ctypes.data_as(C.POINTER(C.c_double))
    _check(load().rs_calibration_fit(n, nf, dp(X), dp(y), dp(r), C.c_double(q), int(max_breakpoints), C.byref(dq), dp(w),
                                     dp(bz), dp(be), C.byref(nbp)), "rs_calibration_fit")
    k = int(nbp.value)
    return float(dq.value), w.tolist(), bz[:k].tolist(), be[:k].tolist()


def rs_cost_table_from_times(cand_ms, pairs):
    """Measured candidate times split over the items in proportion to their pair counts -> int64 nanosecond table."""
    import numpy as np
    ms = np.ascontiguousarray(cand_ms, dtype=np.float64)
    pr = np.ascontiguousarray(pairs, dtype=np.uint64)
    table = np.zeros(pr.shape, dtype=np.int64)
    _check(load().rs_cost_table_from_times(pr.shape[0], pr.shape[1], ms.ctypes.data_as(C.POINTER(C.c_double)),
                                           pr.ctypes.data_as(C.POINTER(C.c_uint64)),
                                           table.ctypes.data_as(C.POINTER(C.c_int64))), "rs_cost_table_from_times")
    return table


def rs_selftest_wait_timeout(status, poll_limit: int = 2000):
    _check(load().rs_selftest_wait_timeout(_ptr(status), C.c_uint(poll_limit), _stream()), "rs_selftest_wait_timeout")


def check_status(status: torch.Tensor, what: str = "kernel"):
    """Reads the device status words (synchronises) and raises if a kernel reported an error."""
    s = status.cpu().tolist()
    if s[0] != 0:
        raise RouteSparseError(f"{what}: device status {s[0]} ({rs_error_string(s[0])}) at site {s[1]}, block {s[2]}")


__all__ = [n for n in dir() if n.startswith(("rs_", "RS_")) or n in
           ("Problem", "IndexSet", "make_library", "new_status", "new_workspace", "check_status", "load", "lib_path",
            "mixture_rows",
            "RouteSparseError", "EXPORTS")]
