"""Seeded synthetic workloads: event streams, T-CSR, replay sets, weights.

This module only *draws inputs*.  It holds none of the model's arithmetic
(no message building, no reductions, no GRU/attention maths); both the CUDA
path and the CPU oracle consume what it produces.

The streams stand in for the public interaction graphs the paper trains on
(Table 2: Wikipedia-, Reddit- and lastfm-shaped node/event counts,
bipartiteness and skew); none of those datasets' records are reproduced.

Recipe (all draws come from counter-based Philox streams keyed by the seed):
  * timestamps: cumulative sum (fp64) of Exp(1) gaps, so t is non-decreasing
    as in the paper's problem statement (Section III-A);
  * endpoints: inverse-CDF lookups in an fp64 Zipf table; bipartite configs
    draw sources from [0, Ns) and destinations from [Ns, N); otherwise both
    from [0, N) with the destination redrawn until it differs from the source;
  * negatives: one per event, uniform over the destination range;
  * edge features ~ N(0, 1): a counter-based integer hash of (seed, eid, col)
    gives twelve 16-bit uniforms whose integer sum (Irwin-Hall) is centred,
    converted to float exactly and scaled by a power of two, so any row can
    be regenerated bit-identically anywhere;
  * auxiliary replay events (mixed batch, Eq. 5): round(rho * B) events drawn
    without replacement from the previous five batches, flagged, merged with
    the B targets and sorted by (t, eid); batch 0 has none;
  * weights: Xavier-uniform matrices, zero biases (optionally small random
    biases for tests), time-encoder frequencies 10^(-9 c / (d - 1)).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    num_nodes: int
    num_src: int            # >0: bipartite, sources [0,num_src), destinations [num_src,N)
    num_events: int
    d_e: int
    feat_dtype: str         # "f32" | "bf16"
    d: int                  # memory = time = embedding dim
    k: int
    heads: int
    batch: int
    replay_frac: float
    prune: bool
    zipf_src: float
    zipf_dst: float
    seed: int

    @property
    def d_msg(self) -> int:
        return 3 * self.d + self.d_e

    @property
    def d_kv(self) -> int:
        return 2 * self.d + self.d_e

    @property
    def num_batches(self) -> int:
        return (self.num_events + self.batch - 1) // self.batch

    @property
    def max_mixed(self) -> int:
        return self.batch + int(round(self.replay_frac * self.batch))


_BASE_SEED = 20260816

CONFIGS: Dict[str, WorkloadConfig] = {
    "tiny": WorkloadConfig("tiny", 1000, 0, 20_000, 16, "f32", 32, 10, 2, 200, 0.0, False, 1.1, 1.1, _BASE_SEED + 0),
    "wiki": WorkloadConfig("wiki", 9000, 8000, 160_000, 172, "f32", 100, 10, 2, 600, 0.0, False, 1.2, 1.0, _BASE_SEED + 1),
    "reddit": WorkloadConfig("reddit", 11000, 10000, 670_000, 172, "f32", 100, 10, 2, 600, 0.2, True, 1.2, 1.0, _BASE_SEED + 2),
    "lastfm": WorkloadConfig("lastfm", 2000, 0, 1_300_000, 0, "f32", 100, 10, 2, 4000, 0.3, True, 1.5, 1.5, _BASE_SEED + 3),
    "large": WorkloadConfig("large", 17000, 0, 50_000_000, 186, "bf16", 100, 10, 2, 4000, 0.2, True, 1.2, 1.2, _BASE_SEED + 4),
}


def scaled(cfg: WorkloadConfig, **kw) -> WorkloadConfig:
    """A copy of a named config with some fields replaced (small test cases)."""
    return replace(cfg, **kw)


# --------------------------------------------------------------------------
# counter-based hashing for edge features
# --------------------------------------------------------------------------
def _mix64(z: np.ndarray) -> np.ndarray:
    """A fixed 64-bit avalanche mixer on uint64 arrays (wrapping arithmetic)."""
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(33)
    z *= np.uint64(0xFF51AFD7ED558CCD)
    z ^= z >> np.uint64(33)
    z *= np.uint64(0xC4CEB9FE1A85EC53)
    z ^= z >> np.uint64(33)
    return z


def edge_feature_rows(seed: int, eids: np.ndarray, d_e: int, dtype: str = "f32") -> np.ndarray:
    """Rows of the edge-feature table for the given event ids.

    Returns float32 [len(eids), d_e] or, for dtype "bf16", uint16 bit
    patterns (round-to-nearest-even of the float32 value).
    """
    eids = np.asarray(eids, dtype=np.uint64).reshape(-1, 1)
    if d_e == 0:
        return np.zeros((eids.shape[0], 0), dtype=np.float32 if dtype == "f32" else np.uint16)
    cols = np.arange(d_e, dtype=np.uint64).reshape(1, -1)
    with np.errstate(over="ignore"):
        base = (np.uint64(seed) * np.uint64(0x9E3779B97F4A7C15)) ^ (eids * np.uint64(0xD1B54A32D192ED03)) ^ (
            cols * np.uint64(0x8CB92BA72F3D8DD7))
        total = np.zeros(base.shape, dtype=np.int64)
        for r in range(3):
            h = _mix64(base + np.uint64(r + 1) * np.uint64(0xA0761D6478BD642F))
            for s in range(4):
                total += ((h >> np.uint64(16 * s)) & np.uint64(0xFFFF)).astype(np.int64)
    centred = 2 * total - 12 * 65535          # |centred| < 2^21: exact in fp32
    x = centred.astype(np.float32) * np.float32(1.0 / 131072.0)
    if dtype == "f32":
        return x
    bits = x.view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def edge_feature_table(cfg: WorkloadConfig, chunk: int = 1 << 18) -> np.ndarray:
    """The whole [E, d_e] table on the host (use only where it fits)."""
    dt = np.float32 if cfg.feat_dtype == "f32" else np.uint16
    out = np.empty((cfg.num_events, cfg.d_e), dtype=dt)
    for e0 in range(0, cfg.num_events, chunk):
        e1 = min(cfg.num_events, e0 + chunk)
        out[e0:e1] = edge_feature_rows(cfg.seed, np.arange(e0, e1), cfg.d_e, cfg.feat_dtype)
    return out


def edge_feature_table_torch(cfg: WorkloadConfig, device, chunk: int = 1 << 20):
    """The same table generated with integer torch ops on `device` (bit-identical)."""
    import torch

    E, de = cfg.num_events, cfg.d_e
    dt = torch.float32 if cfg.feat_dtype == "f32" else torch.bfloat16
    out = torch.empty((E, de), dtype=dt, device=device)
    if de == 0:
        return out

    def s64(v: int) -> int:       # uint64 constant as wrapped int64
        v &= 0xFFFFFFFFFFFFFFFF
        return v - (1 << 64) if v >= (1 << 63) else v

    def lsr(z, n):                # logical shift right on int64 tensors
        return (z >> n) & ((1 << (64 - n)) - 1)

    def mix(z):
        z = z ^ lsr(z, 33)
        z = z * s64(0xFF51AFD7ED558CCD)
        z = z ^ lsr(z, 33)
        z = z * s64(0xC4CEB9FE1A85EC53)
        z = z ^ lsr(z, 33)
        return z

    seed_term = s64(cfg.seed * 0x9E3779B97F4A7C15)
    cols = torch.arange(de, dtype=torch.int64, device=device).view(1, -1) * s64(0x8CB92BA72F3D8DD7)
    for e0 in range(0, E, chunk):
        e1 = min(E, e0 + chunk)
        eids = torch.arange(e0, e1, dtype=torch.int64, device=device).view(-1, 1)
        base = seed_term ^ (eids * s64(0xD1B54A32D192ED03)) ^ cols
        total = torch.zeros_like(base)
        for r in range(3):
            h = mix(base + s64((r + 1) * 0xA0761D6478BD642F))
            for s in range(4):
                total += lsr(h, 16 * s) & 0xFFFF if s else h & 0xFFFF
        centred = 2 * total - 12 * 65535
        x = centred.to(torch.float32) * (1.0 / 131072.0)
        out[e0:e1] = x.to(dt)     # fp32 -> bf16 conversion is round-to-nearest-even
    return out


# --------------------------------------------------------------------------
# event stream
# --------------------------------------------------------------------------
def _zipf_cdf(n: int, s: float) -> np.ndarray:
    w = 1.0 / np.arange(1, n + 1, dtype=np.float64) ** s
    c = np.cumsum(w)
    return c / c[-1]


def _zipf_draw(rng: np.random.Generator, cdf: np.ndarray, size: int) -> np.ndarray:
    u = rng.random(size)
    return np.minimum(np.searchsorted(cdf, u, side="right"), len(cdf) - 1).astype(np.int32)


@dataclass
class EventStream:
    cfg: WorkloadConfig
    src: np.ndarray     # int32 [E]
    dst: np.ndarray     # int32 [E]
    t: np.ndarray       # float64 [E], non-decreasing
    neg: np.ndarray     # int32 [E]
    # T-CSR over both directions of every event, slices sorted by (ts, eid)
    indptr: np.ndarray  # int64 [N+1]
    nbr: np.ndarray     # int32 [2E]
    eid: np.ndarray     # int32 [2E]
    ts: np.ndarray      # float64 [2E]
    _efeat: Optional[np.ndarray] = field(default=None, repr=False)

    def efeat(self) -> np.ndarray:
        if self._efeat is None:
            self._efeat = edge_feature_table(self.cfg)
        return self._efeat


def build_tcsr(src: np.ndarray, dst: np.ndarray, t: np.ndarray, num_nodes: int):
    """Time-sorted adjacency: for every event both (src->dst) and (dst->src)."""
    E = len(src)
    node = np.concatenate([src, dst]).astype(np.int64)
    other = np.concatenate([dst, src]).astype(np.int32)
    eid = np.concatenate([np.arange(E), np.arange(E)]).astype(np.int32)
    ts = np.concatenate([t, t])
    order = np.lexsort((eid, ts, node))       # primary node, then ts, then eid
    counts = np.bincount(node, minlength=num_nodes)
    indptr = np.zeros(num_nodes + 1, dtype=np.int64)
    np.cumsum(counts, out=indptr[1:])
    return indptr, other[order], eid[order], ts[order]


def make_stream(cfg: WorkloadConfig) -> EventStream:
    rng = np.random.Generator(np.random.Philox(key=cfg.seed))
    E, N = cfg.num_events, cfg.num_nodes
    gaps = -np.log1p(-rng.random(E))
    t = np.cumsum(gaps)
    if cfg.num_src > 0:
        ns, nd = cfg.num_src, N - cfg.num_src
        src = _zipf_draw(rng, _zipf_cdf(ns, cfg.zipf_src), E)
        dst = (_zipf_draw(rng, _zipf_cdf(nd, cfg.zipf_dst), E) + ns).astype(np.int32)
        neg = rng.integers(ns, N, size=E, dtype=np.int32)
    else:
        cdf = _zipf_cdf(N, cfg.zipf_src)
        src = _zipf_draw(rng, cdf, E)
        dst = _zipf_draw(rng, _zipf_cdf(N, cfg.zipf_dst), E)
        bad = np.nonzero(dst == src)[0]
        while len(bad):
            dst[bad] = _zipf_draw(rng, cdf, len(bad))
            bad = bad[dst[bad] == src[bad]]
        neg = rng.integers(0, N, size=E, dtype=np.int32)
    indptr, nbr, eid, ts = build_tcsr(src, dst, t, N)
    return EventStream(cfg, src, dst, t, neg, indptr, nbr, eid, ts)


# --------------------------------------------------------------------------
# mixed batches (targets + flagged auxiliary replay events)
# --------------------------------------------------------------------------
@dataclass
class MixedBatch:
    index: int
    src: np.ndarray     # int32 [n]
    dst: np.ndarray     # int32 [n]
    t: np.ndarray       # float64 [n]
    eid: np.ndarray     # int32 [n]
    is_aux: np.ndarray  # uint8 [n]  (1 = auxiliary replay event)

    @property
    def n(self) -> int:
        return len(self.src)


def mixed_batch(stream: EventStream, b: int) -> MixedBatch:
    cfg = stream.cfg
    B = cfg.batch
    lo, hi = b * B, min((b + 1) * B, cfg.num_events)
    tar = np.arange(lo, hi, dtype=np.int64)
    n_rep = int(round(cfg.replay_frac * B)) if b > 0 else 0
    if n_rep > 0:
        pool_lo = max(0, b - 5) * B
        rng = np.random.Generator(np.random.Philox(key=np.array([cfg.seed, b + 1], dtype=np.uint64)))
        rep = pool_lo + rng.choice(lo - pool_lo, size=min(n_rep, lo - pool_lo), replace=False)
        ids = np.concatenate([rep.astype(np.int64), tar])
        aux = np.concatenate([np.ones(len(rep), np.uint8), np.zeros(len(tar), np.uint8)])
    else:
        ids, aux = tar, np.zeros(len(tar), np.uint8)
    order = np.lexsort((ids, stream.t[ids]))
    ids, aux = ids[order], aux[order]
    return MixedBatch(b, stream.src[ids].copy(), stream.dst[ids].copy(), stream.t[ids].copy(),
                      ids.astype(np.int32), aux)


# --------------------------------------------------------------------------
# weights
# --------------------------------------------------------------------------
PARAM_SHAPES = (
    # name, rows (in units resolved below), cols
    "time_w", "time_b", "gru_w_i", "gru_w_h", "gru_b_i", "gru_b_h",
    "w_q", "b_q", "w_k", "w_v", "b_k", "b_v", "w_o", "b_o", "w_1", "b_1", "w_2", "b_2",
)


def param_shapes(d: int, d_e: int, model: str = "tgn") -> Dict[str, tuple]:
    d_msg, d_kv = 3 * d + d_e, 2 * d + d_e
    if model == "jodie":   # plain recurrent cell, time projection (w_p, b_p), the same head
        return {
            "time_w": (d,), "time_b": (d,),
            "rnn_w_i": (d, d_msg), "rnn_w_h": (d, d), "rnn_b_i": (d,), "rnn_b_h": (d,),
            "proj_w": (d,), "proj_b": (d,),
            "w_1": (d, 2 * d), "b_1": (d,), "w_2": (d,), "b_2": (1,),
        }
    return {
        "time_w": (d,), "time_b": (d,),
        "gru_w_i": (3 * d, d_msg), "gru_w_h": (3 * d, d), "gru_b_i": (3 * d,), "gru_b_h": (3 * d,),
        "w_q": (d, 2 * d), "b_q": (d,),
        "w_k": (d, d_kv), "w_v": (d, d_kv), "b_k": (d,), "b_v": (d,),
        "w_o": (d, 2 * d), "b_o": (d,),
        "w_1": (d, 2 * d), "b_1": (d,), "w_2": (d,), "b_2": (1,),
    }


def make_weights(d: int, d_e: int, seed: int, bias_scale: float = 0.0, model: str = "tgn") -> Dict[str, np.ndarray]:
    """Named fp32 tensors; matrices are [out, in] row-major.  The time projection's slope w_p multiplies raw
    time differences (hundreds to thousands of mean gaps), so it is drawn 1000 times smaller than the biases."""
    rng = np.random.Generator(np.random.Philox(key=np.array([seed, 0xBEEF], dtype=np.uint64)))
    out: Dict[str, np.ndarray] = {}
    for name, shape in param_shapes(d, d_e, model).items():
        if name == "time_w":
            c = np.arange(d, dtype=np.float64)
            out[name] = (10.0 ** (-9.0 * c / max(d - 1, 1))).astype(np.float32)
        elif len(shape) == 2:
            a = np.sqrt(6.0 / (shape[0] + shape[1]))
            out[name] = rng.uniform(-a, a, size=shape).astype(np.float32)
        elif name == "w_2":
            a = np.sqrt(6.0 / (shape[0] + 1))
            out[name] = rng.uniform(-a, a, size=shape).astype(np.float32)
        else:
            v = rng.uniform(-bias_scale, bias_scale, size=shape) if bias_scale > 0 else np.zeros(shape)
            out[name] = (v * (1e-3 if name == "proj_w" else 1.0)).astype(np.float32)
    return out
