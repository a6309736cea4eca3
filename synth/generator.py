"""Seeded synthetic Q, K, V with planted attention structure (bf16 bit patterns).

The generator stands in for real Llama-3.1-8B attention inputs on long prompts: the
head geometry (32 query heads, 8 KV heads, d = 128) is the model's, and the planted
structure mirrors the three information topologies the paper names (Section 2.2):
repeated keys that favour vertical columns, locally coherent text that favours a
window / diagonals, and diffuse attention.  None of a benchmark's items or a model's
weights is used.

Recipe (for KV head g shared by its query heads h, unit vector u_g):
    K[g, j] = Kr[g, j] + kboost[j] * gamma0 * u_g + T(j)
    Q[h, i] = Qr[h, i] + gamma_h[i] * u_g + lambda_h[i] * Kr[g, i] + T(i)
    V[g, j] = Vr[g, j]
with Kr, Qr, Vr ~ N(0, 1) i.i.d. from a counter-based generator (Philox keyed by
(seed, layer, tensor, head)), kboost = a_sink on the first four keys and a_vert on the
planted vertical keys, and T an optional rotary-like term on the first 2F dimensions,
T(p) = c_p * (cos(2 pi p / P_f), sin(2 pi p / P_f))_f, whose Q.K contribution depends only
on i - j and decays away from the diagonal.  Everything is computed in float32 and
rounded to bf16 (round to nearest even); both the oracle and the CUDA path consume the
same uint16 bit patterns, so the rounding here is data, not arithmetic of the method.

Only random numbers, planted offsets and dtype conversion live here.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

GAMMA0 = 4.0          # strength of the key-side boost direction
N_SINK_KEYS = 4       # keys 0..3 act as attention sinks
TOEPLITZ_F = 8        # number of rotary-like frequency pairs
_T_Q, _T_K, _T_V, _T_U, _T_MISC, _T_V2, _T_TOPIC = 0, 1, 2, 3, 4, 5, 6


# ----------------------------------------------------------------------------- dtype helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even. NaN is not expected."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _rng(seed: int, layer: int, tensor: int, head: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64((layer << 40) | (tensor << 32) | head)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _normals(seed, layer, tensor, head, shape) -> np.ndarray:
    return _rng(seed, layer, tensor, head).standard_normal(shape, dtype=np.float32)


# ----------------------------------------------------------------------------- specs
@dataclass
class SegmentSpec:
    """Structure planted inside one query/key segment [start, end)."""
    start: int
    end: int
    kind: str = "planted"   # planted | local | delimiter | needle | diffuse


@dataclass
class LayerSpec:
    seed: int
    n: int
    n_q_heads: int
    n_kv_heads: int
    d: int = 128
    layer: int = 0
    gamma: Optional[Sequence[float]] = None      # per query head, mean-query strength
    lam: Optional[Sequence[float]] = None        # per query head, Q_i += lam * Kr_i
    a_sink: Optional[Sequence[float]] = None     # per KV head
    a_vert: Optional[Sequence[float]] = None     # per KV head
    n_vert: int = 8
    toeplitz: bool = True
    toeplitz_boost: object = 6.0                 # logit boost on the diagonal from T (float, or one per query head)
    toeplitz_periods: Optional[Sequence[float]] = None   # (shortest, longest) period; default (512, 8 n)
    toeplitz_f: int = TOEPLITZ_F                 # number of frequency pairs (first 2 F dimensions)
    disjoint_dims: bool = False                  # keep the planted directions out of the rotary dimensions
    q_noise: Optional[Sequence[float]] = None    # per query head, scale of the unstructured part Qr (1 = literal)
    nu: Optional[Sequence[float]] = None         # per query head, response to planted verticals along a second
                                                 # direction v_g (None: verticals share the sink direction u_g)
    topic_q: Optional[Sequence[float]] = None    # per query head, strength of the chunk-topic component
    topic_k: Optional[Sequence[float]] = None    # per KV head, strength of the chunk-topic component
    n_topics: int = 24
    topic_chunk: int = 256
    segments: List[SegmentSpec] = field(default_factory=list)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def seg_bounds(self) -> List[int]:
        if not self.segments:
            return [0, self.n]
        return [s.start for s in self.segments] + [self.segments[-1].end]


def tiny_spec(seed: int, n: int, n_q_heads: int = 2, n_kv_heads: int = 1, d: int = 128,
              toeplitz: bool = True, n_vert: int = 3) -> LayerSpec:
    """Small layer for unit tests (same recipe, per-head strengths drawn from the seed)."""
    r = _rng(seed, 0, _T_MISC, 1000)
    return LayerSpec(seed=seed, n=n, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, d=d,
                     gamma=r.uniform(2.0, 6.0, n_q_heads).tolist(),
                     lam=r.uniform(0.25, 0.75, n_q_heads).tolist(),
                     a_sink=r.uniform(2.0, 6.0, n_kv_heads).tolist(),
                     a_vert=r.uniform(1.5, 4.5, n_kv_heads).tolist(),
                     n_vert=n_vert, toeplitz=toeplitz)


def config1_spec(toeplitz: bool = False, n: int = 4096) -> LayerSpec:
    """Single head, n = 4096: sinks on keys 0-3 (strength 4), 8 planted verticals (3), local 0.5."""
    return LayerSpec(seed=260829058 + 1, n=n, n_q_heads=1, n_kv_heads=1,
                     gamma=[4.0], lam=[0.5], a_sink=[4.0], a_vert=[3.0], n_vert=8, toeplitz=toeplitz)


def config2_spec(n: int = 32768, seed_offset: int = 2, n_q_heads: int = 32, n_kv_heads: int = 8) -> LayerSpec:
    """Llama-3.1-8B-shaped layer with per-head random sink / vertical / local strengths."""
    seed = 260829058 + seed_offset
    r = _rng(seed, 0, _T_MISC, 1001)
    return LayerSpec(seed=seed, n=n, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                     gamma=r.uniform(2.0, 6.0, n_q_heads).tolist(),
                     lam=r.uniform(0.25, 0.75, n_q_heads).tolist(),
                     a_sink=r.uniform(2.0, 6.0, n_kv_heads).tolist(),
                     a_vert=r.uniform(1.5, 4.5, n_kv_heads).tolist(),
                     n_vert=8, toeplitz=True)


def config3_spec(n: int = 131072, seed_offset: int = 3, n_q_heads: int = 32, n_kv_heads: int = 8) -> LayerSpec:
    """Llama-3.1-8B-shaped layer whose heads follow four archetypes, with boosts that grow with log(n) so that the
    mass split between structure and the diffuse background stays what it is at n = 4096:
      local/sink heads (window + initial tokens), vertical heads (planted columns), topic heads (separated key
      blocks of the same topic as the query's chunk) and diffuse heads (little structure: dense fallback).
    Archetypes are dealt to the heads of every KV group by a seeded permutation."""
    seed = 260829058 + seed_offset
    r = _rng(seed, 0, _T_MISC, 1004)
    sd, comp = np.sqrt(128.0), np.log(max(n, 4096) / 4096.0)
    G = n_q_heads // n_kv_heads
    kinds = []
    for g in range(n_kv_heads):
        base = ["local", "vertical", "topic", "local" if g % 2 == 0 else "vertical"][:G] if G <= 4 else ["local", "vertical", "topic"] * G
        base = list(base[:G])
        if g % 3 == 2 and G >= 2:
            base[-1] = "diffuse"
        kinds += [base[i] for i in r.permutation(G)]
    # Log-weights (natural log of a component's total unnormalised softmax weight) relative to a top level w_top;
    # the diffuse background has log-weight ~ ln(n) + 0.5.  Sinks: 4 keys, verticals: 8 keys, topic: ~ n / (2 T) keys.
    gamma0_k = 4.0                                   # query-side response that realises the key-side base logit
    w_top = 14.5
    B_s = [w_top - np.log(4.0) + r.uniform(-0.3, 0.3) + comp for _ in range(n_kv_heads)]     # key-side base logits
    B_v = [w_top - np.log(8.0) + r.uniform(-0.3, 0.3) + comp for _ in range(n_kv_heads)]
    B_t = [w_top - 4.4 + r.uniform(-0.3, 0.3) for _ in range(n_kv_heads)]                    # key count grows with n
    a_sink = [b * sd / (GAMMA0 * gamma0_k) for b in B_s]
    a_vert = [b * sd / (GAMMA0 * gamma0_k) for b in B_v]
    topic_k = [float(np.sqrt(b * sd)) for b in B_t]
    # per archetype: offsets below the top level for (sink, vertical, local, topic)
    drop = {"local": (0.5, 6.0, 0.0, None), "vertical": (0.5, 0.0, 0.5, None), "topic": (2.0, 6.0, 1.0, 0.0),
            "diffuse": (7.0, 8.0, 7.0, None)}
    gamma, nu, lam, qn, tq, tb = [], [], [], [], [], []
    for h, kind in enumerate(kinds):
        g = h // G
        ds, dv, dl, dt = drop[kind]
        jit = lambda: r.uniform(-0.25, 0.25)
        lam_h = 0.5 if kind == "diffuse" else r.uniform(0.1, 0.3)
        gamma.append(gamma0_k * (B_s[g] - ds + jit()) / B_s[g])
        nu.append(gamma0_k * (B_v[g] - dv + jit()) / B_v[g])
        tb.append(w_top - dl - lam_h * sd - 0.7 + comp + jit())
        tq.append(0.0 if dt is None else topic_k[g] * (B_t[g] - dt + jit()) / B_t[g])
        lam.append(lam_h)
        qn.append(1.0 if kind == "diffuse" else 0.25)
    spec = LayerSpec(seed=seed, n=n, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, gamma=gamma, lam=lam,
                     a_sink=a_sink, a_vert=a_vert, n_vert=8, toeplitz=True, toeplitz_boost=tb,
                     toeplitz_periods=(37.0, 5300.0), toeplitz_f=28, disjoint_dims=True, q_noise=qn, nu=nu, topic_q=tq, topic_k=topic_k)
    spec.kinds = kinds
    return spec


def config4_layer_spec(layer: int, n: int = 131072, seg_len: int = 32768,
                       n_q_heads: int = 32, n_kv_heads: int = 8) -> LayerSpec:
    """One layer of the segmented stack: structure switches every seg_len tokens, order seeded per layer."""
    spec = config3_spec(n=n, seed_offset=4, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads)
    spec.layer = layer
    kinds = ["local", "delimiter", "needle", "diffuse"]
    order = _rng(spec.seed, layer, _T_MISC, 1002).permutation(len(kinds))
    n_seg = n // seg_len
    spec.segments = [SegmentSpec(s * seg_len, (s + 1) * seg_len, kinds[order[s % len(kinds)]])
                     for s in range(n_seg)]
    return spec


def fixed_routes_config2(n_q_heads: int = 32, seed: int = 260829058 + 2) -> np.ndarray:
    """Seeded head -> pattern assignment: 30% A-shape, 30% vertical-slash, 30% block-sparse, 10% dense.

    Returns int32[n_q_heads] with values 1 (A-shape), 2 (vertical-slash), 3 (block-sparse), 0 (dense).
    Counts are rounded down and leftovers go to A-shape, then vertical-slash (10/10/9/3 of 32).
    """
    n_a = int(0.3 * n_q_heads)
    n_v = int(0.3 * n_q_heads)
    n_b = int(0.3 * n_q_heads)
    n_d = max(1, int(0.1 * n_q_heads)) if n_q_heads >= 4 else 0
    left = n_q_heads - (n_a + n_v + n_b + n_d)
    for _ in range(left):
        if n_a <= n_v:
            n_a += 1
        else:
            n_v += 1
    labels = np.array([1] * n_a + [2] * n_v + [3] * n_b + [0] * n_d, dtype=np.int32)
    perm = _rng(seed, 0, _T_MISC, 1003).permutation(n_q_heads)
    out = np.empty(n_q_heads, dtype=np.int32)
    out[perm] = labels
    return out


# ----------------------------------------------------------------------------- generation
def _toeplitz_table(n: int, d: int, boost: float, period_range=None, F: int = TOEPLITZ_F) -> np.ndarray:
    """[n, 2F] float32 rows c * (cos, sin)(2 pi p / P_f); c^2 * F / sqrt(d) = boost."""
    c = np.sqrt(boost * np.sqrt(d) / F)
    lo, hi = period_range if period_range is not None else (512.0, 8.0 * n)
    periods = np.geomspace(float(lo), float(hi), F)
    pos = np.arange(n, dtype=np.float64)[:, None]
    ang = 2.0 * np.pi * pos / periods[None, :]
    t = np.empty((n, 2 * F), dtype=np.float32)
    t[:, 0::2] = (c * np.cos(ang)).astype(np.float32)
    t[:, 1::2] = (c * np.sin(ang)).astype(np.float32)
    return t


def make_layer(spec: LayerSpec, heads: Optional[Sequence[int]] = None) -> Dict[str, np.ndarray]:
    """Generate bf16 bit patterns Q[Hq, n, d], K[Hkv, n, d], V[Hkv, n, d] (uint16) for one layer.

    `heads` optionally restricts the query heads generated (their KV heads are generated as
    needed); the returned Q then has len(heads) rows in that order and K, V keep all KV heads
    that were touched (others zero).  Meta data: planted vertical positions per KV head.
    """
    n, d, Hq, Hkv = spec.n, spec.d, spec.n_q_heads, spec.n_kv_heads
    G = spec.group
    gamma = np.asarray(spec.gamma if spec.gamma is not None else [4.0] * Hq, dtype=np.float32)
    lam = np.asarray(spec.lam if spec.lam is not None else [0.5] * Hq, dtype=np.float32)
    a_sink = np.asarray(spec.a_sink if spec.a_sink is not None else [4.0] * Hkv, dtype=np.float32)
    a_vert = np.asarray(spec.a_vert if spec.a_vert is not None else [3.0] * Hkv, dtype=np.float32)
    q_heads = list(range(Hq)) if heads is None else list(heads)
    kv_needed = sorted({h // G for h in q_heads})

    segs = spec.segments or [SegmentSpec(0, n, "planted")]
    tb_heads = np.broadcast_to(np.asarray(spec.toeplitz_boost, dtype=np.float64), (Hq,))
    tb_mean = float(tb_heads.mean())     # the key side carries the mean boost, each query head rescales its side
    # per-position modifiers shared by all heads
    lam_scale = np.ones(n, dtype=np.float32)      # multiplies lambda_h
    lam_abs = np.full(n, -1.0, dtype=np.float32)  # >= 0 overrides lambda_h
    gam_scale = np.ones(n, dtype=np.float32)
    tz_amp = np.ones(n, dtype=np.float32) if spec.toeplitz else np.zeros(n, dtype=np.float32)
    for s in segs:
        sl = slice(s.start, s.end)
        if s.kind == "local":
            lam_abs[sl] = 1.0
            tz_amp[sl] = np.sqrt(8.0 / tb_mean) if spec.toeplitz else 0.0
        elif s.kind == "diffuse":
            lam_scale[sl] = 0.0
            gam_scale[sl] = 0.0
            tz_amp[sl] = 0.0
    ttab = _toeplitz_table(n, d, tb_mean, spec.toeplitz_periods, spec.toeplitz_f) if tz_amp.any() else None
    TF2 = 2 * spec.toeplitz_f

    Q = np.zeros((len(q_heads), n, d), dtype=np.uint16)
    K = np.zeros((Hkv, n, d), dtype=np.uint16)
    V = np.zeros((Hkv, n, d), dtype=np.uint16)
    vert_pos: Dict[int, np.ndarray] = {}
    kr_cache: Dict[int, np.ndarray] = {}
    u_cache: Dict[int, np.ndarray] = {}
    needle_cache: Dict[int, Dict[str, np.ndarray]] = {}
    v_cache: Dict[int, np.ndarray] = {}
    topic_cache: Dict[int, np.ndarray] = {}

    for g in kv_needed:
        u = _normals(spec.seed, spec.layer, _T_U, g, (d,)).astype(np.float64)
        if spec.disjoint_dims:
            u[:TF2] = 0.0
        u = (u / np.linalg.norm(u)).astype(np.float32)
        u_cache[g] = u
        Kr = _normals(spec.seed, spec.layer, _T_K, g, (n, d))
        rg = _rng(spec.seed, spec.layer, _T_MISC, g)
        kboost = np.zeros(n, dtype=np.float32)
        planted: List[int] = []
        needles: Dict[str, np.ndarray] = {}
        for si, s in enumerate(segs):
            L = s.end - s.start
            if s.kind == "planted":
                if s.start == 0:
                    kboost[:min(N_SINK_KEYS, n)] = a_sink[g]
                lo, hi = s.start + N_SINK_KEYS, max(s.start + N_SINK_KEYS + 1, s.end - 64)
                k = min(spec.n_vert, max(0, hi - lo))
                pos = np.sort(rg.choice(np.arange(lo, hi), size=k, replace=False)) if k > 0 else np.zeros(0, int)
                kboost[pos] = a_vert[g]
                planted += pos.tolist()
            elif s.kind == "delimiter":
                pos = np.arange(s.start, s.end, 257)
                kboost[pos] = a_vert[g] if spec.nu is not None else 4.0
                planted += pos.tolist()
            elif s.kind == "needle":
                # 16 key vectors, each copied to 8 seeded positions of the segment
                nv = rg.standard_normal((16, d), dtype=np.float32)
                pos = rg.choice(np.arange(s.start, max(s.start + 1, s.end - 64)), size=min(128, max(1, L - 64)),
                                replace=False)
                for t, p in enumerate(pos):
                    Kr[p] = nv[t % 16]
                needles[str(si)] = nv
                planted += np.sort(pos).tolist()
        needle_cache[g] = needles
        vert_pos[g] = np.asarray(sorted(planted), dtype=np.int64)
        kr_cache[g] = Kr
        if spec.nu is not None:          # verticals along a second direction, sinks along u
            v2 = _normals(spec.seed, spec.layer, _T_V2, g, (d,)).astype(np.float64)
            if spec.disjoint_dims:
                v2[:TF2] = 0.0
            v2 = v2 - (v2 @ u.astype(np.float64)) * u.astype(np.float64)
            v2 = (v2 / np.linalg.norm(v2)).astype(np.float32)
            v_cache[g] = v2
            sink_part = np.zeros(n, dtype=np.float32)
            sink_part[:min(N_SINK_KEYS, n)] = kboost[:min(N_SINK_KEYS, n)]
            vert_part = kboost - sink_part
            Kf = Kr + (sink_part * GAMMA0)[:, None] * u[None, :] + (vert_part * GAMMA0)[:, None] * v2[None, :]
        else:
            Kf = Kr + (kboost * GAMMA0)[:, None] * u[None, :]
        if spec.topic_k is not None:
            rt = _rng(spec.seed, spec.layer, _T_TOPIC, g)
            E = rt.standard_normal((spec.n_topics, d), dtype=np.float32)
            if spec.disjoint_dims:
                E[:, :TF2] = 0.0
            E /= np.linalg.norm(E, axis=1, keepdims=True)
            n_chunks = (n + spec.topic_chunk - 1) // spec.topic_chunk
            topic_of_pos = np.repeat(rt.integers(0, spec.n_topics, n_chunks), spec.topic_chunk)[:n]
            topic_cache[g] = E[topic_of_pos]
            Kf += np.float32(spec.topic_k[g]) * topic_cache[g]
        if ttab is not None:
            Kf[:, :TF2] += tz_amp[:, None] * ttab
        K[g] = f32_to_bf16_bits(Kf)
        V[g] = f32_to_bf16_bits(_normals(spec.seed, spec.layer, _T_V, g, (n, d)))

    for qi, h in enumerate(q_heads):
        g = h // G
        Qr = _normals(spec.seed, spec.layer, _T_Q, h, (n, d))
        lam_pos = np.where(lam_abs >= 0, lam_abs, lam[h] * lam_scale).astype(np.float32)
        if spec.q_noise is not None:
            Qr = Qr * np.float32(spec.q_noise[h])
        Qf = Qr + (gamma[h] * gam_scale)[:, None] * u_cache[g][None, :] + lam_pos[:, None] * kr_cache[g]
        if spec.nu is not None:
            Qf += (np.float32(spec.nu[h]) * gam_scale)[:, None] * v_cache[g][None, :]
        if spec.topic_q is not None and spec.topic_k is not None:
            Qf += np.float32(spec.topic_q[h]) * topic_cache[g]
        if ttab is not None:
            Qf[:, :TF2] += (np.float32(tb_heads[h] / tb_mean) * tz_amp)[:, None] * ttab
        for si, s in enumerate(segs):
            if s.kind == "needle" and str(si) in needle_cache[g]:
                nv = needle_cache[g][str(si)]
                rows = np.arange(max(s.start, s.end - 64), s.end)
                Qf[rows] += 0.5 * nv[rows % 16]
        Q[qi] = f32_to_bf16_bits(Qf)

    return {"Q": Q, "K": K, "V": V, "vert_pos": vert_pos, "q_heads": np.asarray(q_heads),
            "seg_bounds": np.asarray(spec.seg_bounds(), dtype=np.int32)}
