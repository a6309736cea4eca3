"""Helpers shared by the GPU parity tests: upload of seeded inputs and of oracle-built index sets."""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np
import torch

import paper_2608_29058_b200 as rs
from oracle import patterns as PT
from oracle import probe as OP
from synth import bf16_bits_to_f64

ATOL_MAX, ATOL_MEAN = 2e-2, 5e-3      # attention output vs the oracle under the same mask


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def f64_heads(L: Dict[str, np.ndarray]):
    return ([bf16_bits_to_f64(x) for x in L["Q"]], [bf16_bits_to_f64(x) for x in L["K"]],
            [bf16_bits_to_f64(x) for x in L["V"]])


def c_library(cands: Sequence[PT.Candidate]):
    return rs.make_library([(c.pattern, c.b0, c.b1, 0) for c in cands])


def oracle_probe_all(Qs, Ks, p: rs.Problem):
    """Oracle probe for every (segment, head): dict item -> (ProbeResult, bscore)."""
    out = {}
    G = p.n_q_heads // p.n_kv_heads
    for s in range(p.n_segments):
        q0, q1 = p.seg_bounds[s], p.seg_bounds[s + 1]
        for h in range(p.n_q_heads):
            pr = OP.probe_rows(Qs[h], Ks[h // G], q1)
            bs = OP.block_scores(Qs[h], Ks[h // G], q0, q1)
            out[s * p.n_q_heads + h] = (pr, bs)
    return out


def oracle_index_sets(p: rs.Problem, cands: Sequence[PT.Candidate], choice: Sequence[int], probes) -> List[PT.IndexSet]:
    sets = []
    for item in range(p.n_items):
        s = item // p.n_q_heads
        pr, bs = probes[item]
        sets.append(PT.build_indices(cands[choice[item]], p.seg_bounds[s], p.seg_bounds[s + 1], pr.vert, pr.slash, bs))
    return sets


def upload_materialised(p: rs.Problem, lib, sets: List[PT.IndexSet]) -> rs.IndexSet:
    idx = rs.IndexSet.for_library(p, lib, materialised=True)
    nb = p.n_keys // 64
    vs_cols = idx.vs_cols.cpu().numpy(); vs_offs = idx.vs_offs.cpu().numpy()
    vs_diag = idx.vs_diag.cpu().numpy(); vs_count = idx.vs_count.cpu().numpy()
    bs_blk = idx.bs_blk.cpu().numpy(); bs_count = idx.bs_count.cpu().numpy()
    for item, ix in enumerate(sets):
        h = item % p.n_q_heads
        if ix.cand.pattern == PT.VERTICAL_SLASH:
            vs_cols[item, :len(ix.V)] = ix.V; vs_offs[item, :len(ix.S)] = ix.S; vs_diag[item, :len(ix.D)] = ix.D
            vs_count[item] = [len(ix.V), len(ix.S), len(ix.D), 0]
        elif ix.cand.pattern == PT.BLOCK_SPARSE:
            for t, sel in enumerate(ix.blk):
                row = h * nb + ix.q0 // 64 + t
                bs_blk[row, :len(sel)] = sel
                bs_count[row] = len(sel)
    for name, arr in (("vs_cols", vs_cols), ("vs_offs", vs_offs), ("vs_diag", vs_diag), ("vs_count", vs_count),
                      ("bs_blk", bs_blk), ("bs_count", bs_count)):
        getattr(idx, name).copy_(torch.from_numpy(arr))
    return idx


def assert_attention_close(O_gpu: np.ndarray, O_ref: np.ndarray, what=""):
    err = np.abs(O_gpu.astype(np.float64) - O_ref.astype(np.float64))
    assert not np.isnan(O_gpu).any(), what
    assert err.max() <= ATOL_MAX, f"{what}: max-abs {err.max():.3e}"
    assert err.mean() <= ATOL_MEAN, f"{what}: mean-abs {err.mean():.3e}"
