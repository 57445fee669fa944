"""Seeded input generators (numpy, counter-based Philox streams).

Every tensor is drawn in independent blocks of ``BLOCK`` rows whose stream key
is (seed, tensor id, layer, sequence, block index), so any row range of any
tensor can be produced on its own, bit-identically, without drawing the rows
before it.  Values are drawn in fp32 and rounded once to bf16
(round-to-nearest-even); tensors are returned as ``uint16`` bf16 bit patterns.

Nothing here performs a step of the method itself.  The planted-needle
workload multiplies a query-cluster centre through the two random compressor
matrices only to *construct a key vector* whose compressed image lines up with
that cluster's compressed image; the method's own compression, scoring and
selection are never run here.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from functools import lru_cache
import os

import numpy as np

from .configs import EsaShape

BLOCK = 1024
_TID = {"q": 1, "k": 2, "v": 3, "wq": 4, "wk": 5, "hscale": 6, "ck": 7, "cq": 8,
        "zk": 9, "zq": 10, "plan": 11, "bias": 12}

# planted-needle recipe constants (config "gmm_needles")
N_CENTRES = 64
CLUSTER_STD = 0.3
N_SPANS = 32
SPAN_LEN = 16
ALIGNED_QUERIES = 16      # queries per aligned chunk forced into the span's cluster
NEEDLE_GAIN = 2.0         # gamma: length of the planted key direction
NEEDLE_STD = 0.05         # per-token noise on a planted key


def _rng(seed: int, *ids: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), *map(int, ids)])))


# ----------------------------------------------------------------------------
# dtype plumbing (representation only)
# ----------------------------------------------------------------------------
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern (uint16), round-to-nearest-even.  Finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------
# plain normal tensors
# ----------------------------------------------------------------------------
def _normal_block(seed, ids, blk, ncols) -> np.ndarray:
    return _rng(seed, *ids, blk).standard_normal((BLOCK, ncols), dtype=np.float32)


def _blocks(row0: int, row1: int):
    for blk in range(row0 // BLOCK, (row1 + BLOCK - 1) // BLOCK):
        lo = max(row0, blk * BLOCK)
        hi = min(row1, (blk + 1) * BLOCK)
        yield blk, lo, hi


def _parallel(fn, items):
    items = list(items)
    nthr = min(len(items), max(1, (os.cpu_count() or 1)))
    if nthr <= 1:
        return [fn(it) for it in items]
    with ThreadPoolExecutor(nthr) as ex:
        return list(ex.map(fn, items))


def normal_bf16(seed: int, ids, row0: int, row1: int, ncols: int, col_scale=None) -> np.ndarray:
    """Rows [row0,row1) of an N(0,1) matrix with ``ncols`` columns, optionally
    scaled per column, as bf16 bits [row1-row0, ncols]."""
    out = np.empty((row1 - row0, ncols), dtype=np.uint16)

    def work(item):
        blk, lo, hi = item
        x = _normal_block(seed, ids, blk, ncols)[lo - blk * BLOCK: hi - blk * BLOCK]
        if col_scale is not None:
            x = x * col_scale
        out[lo - row0: hi - row0] = to_bf16_bits(x)

    _parallel(work, _blocks(row0, row1))
    return out


def compressor_weights(cfg: EsaShape, layer: int = 0):
    """fp32 compressor matrices: Wq [d_c, d_H] ~ N(0, 1/d_H), Wk [d_c, d_G] ~ N(0, 1/d_G)."""
    wq = _rng(cfg.seed, _TID["wq"], layer).standard_normal((cfg.d_c, cfg.d_H), dtype=np.float32)
    wk = _rng(cfg.seed, _TID["wk"], layer).standard_normal((cfg.d_c, cfg.d_G), dtype=np.float32)
    wq *= np.float32(1.0 / np.sqrt(cfg.d_H))
    wk *= np.float32(1.0 / np.sqrt(cfg.d_G))
    return wq, wk


def compressor_bias(cfg: EsaShape, layer: int = 0):
    """Optional fp32 biases (unit tests only; the five workloads use none)."""
    g = _rng(cfg.seed, _TID["bias"], layer)
    return (g.standard_normal(cfg.d_c, dtype=np.float32),
            g.standard_normal(cfg.d_c, dtype=np.float32))


def _head_scale(cfg: EsaShape, which: str, layer: int, seq: int) -> np.ndarray:
    nh = cfg.H if which == "q" else cfg.H_G
    s = _rng(cfg.seed, _TID["hscale"], _TID[which], layer, seq).uniform(0.5, 2.0, size=nh)
    return np.repeat(s.astype(np.float32), cfg.d)


# ----------------------------------------------------------------------------
# planted needles (mixture keys, spans aligned to a later query cluster)
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class NeedlePlan:
    span_start: np.ndarray      # [N_SPANS] first token of each planted span
    span_len: int
    aligned_chunk: np.ndarray   # [N_SPANS] index of the chunk whose queries look for span i
    q_cluster: np.ndarray       # [N_SPANS] query-mixture component the span is aligned to
    aligned_rows: dict = field(default_factory=dict)  # token position -> forced query cluster
    centres_k: np.ndarray = None  # [N_CENTRES, d_G] fp32
    centres_q: np.ndarray = None  # [N_CENTRES, d_H] fp32
    directions: np.ndarray = None  # [N_SPANS, d_G] fp32 planted key directions (already scaled)

    def spans_in_chunk(self, chunk: int):
        return [i for i in range(len(self.span_start)) if int(self.aligned_chunk[i]) == chunk]

    def needle_tokens(self, i: int) -> np.ndarray:
        return np.arange(int(self.span_start[i]), int(self.span_start[i]) + self.span_len)


@lru_cache(maxsize=8)
def needle_plan(cfg: EsaShape, layer: int = 0) -> NeedlePlan:
    """Where the needle spans sit, which later chunk asks for each, and the
    planted key directions, for one layer of a ``gmm_needles`` workload."""
    assert cfg.kind == "gmm_needles"
    g = _rng(cfg.seed, _TID["plan"], layer)
    ck = _rng(cfg.seed, _TID["ck"], layer).standard_normal((N_CENTRES, cfg.d_G), dtype=np.float32)
    cq = _rng(cfg.seed, _TID["cq"], layer).standard_normal((N_CENTRES, cfg.d_H), dtype=np.float32)
    lo, hi = cfg.l_I, cfg.S - cfg.l_L - 2 * cfg.l_C
    assert hi - lo >= N_SPANS * 4 * SPAN_LEN, "context too short for the needle recipe"
    stride = (hi - lo) // N_SPANS
    n_chunks = cfg.S // cfg.l_C
    span_start = np.empty(N_SPANS, dtype=np.int64)
    aligned = np.empty(N_SPANS, dtype=np.int64)
    q_cluster = g.permutation(N_CENTRES)[:N_SPANS].astype(np.int64)
    rows = {}
    for i in range(N_SPANS):
        p = lo + i * stride + int(g.integers(0, stride - SPAN_LEN))
        span_start[i] = p
        # first chunk start t with the span inside M = [l_I, t - l_L) and l_M > k
        t_min = max(p + SPAN_LEN + cfg.l_L, cfg.l_I + cfg.l_L + cfg.k + 1)
        c_min = -(-t_min // cfg.l_C)
        c = int(g.integers(c_min, n_chunks))
        aligned[i] = c
        offs = g.permutation(cfg.l_C)[:ALIGNED_QUERIES]
        for o in offs:
            rows[c * cfg.l_C + int(o)] = int(q_cluster[i])
    wq, wk = compressor_weights(cfg, layer)
    # planted direction: gamma * Wk^T (Wq q*), q* = the aligned query-cluster centre
    dirs = np.empty((N_SPANS, cfg.d_G), dtype=np.float32)
    for i in range(N_SPANS):
        qstar = cq[q_cluster[i]].astype(np.float64)
        dirs[i] = (NEEDLE_GAIN * (wk.astype(np.float64).T @ (wq.astype(np.float64) @ qstar))).astype(np.float32)
    return NeedlePlan(span_start, SPAN_LEN, aligned, q_cluster, rows, ck, cq, dirs)


def _gmm_rows(cfg: EsaShape, which: str, layer: int, seq: int, row0: int, row1: int) -> np.ndarray:
    plan = needle_plan(cfg, layer)
    ncols = cfg.d_H if which == "q" else cfg.d_G
    centres = plan.centres_q if which == "q" else plan.centres_k
    ztid = _TID["zq"] if which == "q" else _TID["zk"]
    out = np.empty((row1 - row0, ncols), dtype=np.uint16)

    def work(item):
        blk, lo, hi = item
        z = _rng(cfg.seed, ztid, layer, seq, blk).integers(0, N_CENTRES, size=BLOCK)
        noise = _normal_block(cfg.seed, (_TID[which], layer, seq), blk, ncols)
        base = blk * BLOCK
        if which == "q":
            for pos, cl in plan.aligned_rows.items():
                if base <= pos < base + BLOCK:
                    z[pos - base] = cl
            x = centres[z] + np.float32(CLUSTER_STD) * noise
        else:
            x = centres[z] + np.float32(CLUSTER_STD) * noise
            for i in range(len(plan.span_start)):
                p0 = int(plan.span_start[i])
                a, b = max(p0, base), min(p0 + plan.span_len, base + BLOCK)
                if a < b:
                    x[a - base: b - base] = plan.directions[i] + np.float32(NEEDLE_STD) * noise[a - base: b - base]
        out[lo - row0: hi - row0] = to_bf16_bits(x[lo - base: hi - base])

    _parallel(work, _blocks(row0, row1))
    return out


# ----------------------------------------------------------------------------
# public: rows of Q / K / V
# ----------------------------------------------------------------------------
def qkv_rows(cfg: EsaShape, which: str, row0: int, row1: int, layer: int = 0, seq: int = 0) -> np.ndarray:
    """Token rows [row0,row1) of tensor ``which`` in {"q","k","v"} for one layer
    and sequence, as bf16 bits shaped [rows, heads, d] (heads = H for q, H_G for k/v)."""
    assert which in ("q", "k", "v") and 0 <= row0 <= row1
    nh = cfg.H if which == "q" else cfg.H_G
    ncols = nh * cfg.d
    if cfg.kind == "gmm_needles" and which in ("q", "k"):
        x = _gmm_rows(cfg, which, layer, seq, row0, row1)
    else:
        scale = _head_scale(cfg, which, layer, seq) if cfg.kind == "headscale" else None
        x = normal_bf16(cfg.seed, (_TID[which], layer, seq), row0, row1, ncols, scale)
    return x.reshape(row1 - row0, nh, cfg.d)
