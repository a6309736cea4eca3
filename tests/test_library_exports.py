"""CPU-side checks of the boundary: the C-ABI library loads and exports every symbol the header declares."""
import ctypes
import os
import re

import paper_2608_29058_b200 as rs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "routesparse.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rs_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = rs.load()
    names = declared_symbols()
    assert {"rs_probe", "rs_build_indices", "rs_route", "rs_sparse_prefill_attn", "rs_certificate",
            "rs_dense_prefill_attn", "rs_workspace_bytes"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(rs.EXPORTS) == set(names)


def test_host_side_calls_without_a_gpu():
    assert rs.rs_version() >= 100
    assert "workspace" in rs.rs_error_string(-3)
    p = rs.Problem(32, 8, 131072)
    lib = rs.make_library(rs.default_library())
    assert rs.rs_workspace_bytes(p, lib) > 32 * 2048 * 2048 * 4        # fused block scores dominate
    assert rs.rs_workspace_bytes(p, None) < 64 << 20
    for bad in (rs.Problem(32, 8, 100), rs.Problem(32, 5, 128), rs.Problem(32, 8, 256, [0, 100, 256]),
                rs.Problem(32, 8, 128, [0, 64]), rs.Problem(32, 8, 256, head_dim=64)):
        try:
            rs.rs_workspace_bytes(bad, None)
            assert False, "expected an error"
        except rs.RouteSparseError:
            pass


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(rs.rs_candidate) == 16
    assert ctypes.sizeof(rs.rs_route_params) == 120
    assert ctypes.sizeof(rs.rs_index_set) == 24 + 6 * 8
    assert rs.rs_route_params.forced_dense.offset == 56


def test_budget_helpers():
    assert rs.dense_flops([0, 4096], 1) == 4 * 128 * (4096 * 4097 // 2)
    assert rs.probe_flops([0, 128], 2) == 2 * 64 * 128 * 128 * 2 + 2 * 128 * 2 * 3
