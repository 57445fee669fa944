"""CPU oracle for one step of Efficient Selective Attention (ESA).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
select-plus-attend step computes, written from the paper's equations in numpy
float64.  It shares no code with the CUDA library and must never be imported
by it; only the tests, the smoke check and the benchmark's CPU-baseline leg
call it.

Paper notation: H query heads, H_G key/value heads, d head dim, d_H = H*d,
d_G = H_G*d, d' = d_c compressed dim; the tokens before the current chunk C
(t of them) split into initial I, middle M, local L (Section 3.1).

Step, in the paper's order:
  partition            Section 3.1            I = [0,i_end), M = [i_end,m_end), L = [m_end,t)
  compress             Eq. 5                  q' = f_q(q), k' = f_k(k): one linear layer each
  scores               Eq. 6                  S[c,m] = q'_c . k'_m
  aggregate            Eq. 4                  s_m = max_c ( S[c,m] - max_m' S[c,m'] )
  proximity_pool       Eq. 8                  s'_j = max of s over [j-eps, j+eps] clipped to M
  topk                 Eq. 2                  k largest s', ties to the lowest index
  attend               Eq. 1 / Algorithm 1    softmax attention over I u M_k u L u C (C causal)

Precision (the paper states none; these are the readings the library follows):
compressor weights are rounded once to bf16; q' and k' are accumulated exactly
(float64 here) and rounded to bf16; S is rounded to fp32 and Eq. 4 / Eq. 8 run
in fp32; attention runs in float64 on the bf16 inputs.

Pins (tests/test_oracle_pins.py): attention == textbook causal attention when
k >= l_M; part-by-part attention merged by log-normalisers (Algorithm 1) == one
softmax over the union, also with distinct far/near queries and keys (Section 3.2);
scores/aggregate/top-k == brute-force loops on tiny inputs; proximity_pool ==
a library 1-D max pool; compress == plain matrix product and the GQA folding
identity; the flop/cache closed forms reproduce the paper's 1.56 % and 6.25 %.
The paper prints no worked numeric example, so absolute output values are
"parity unpinned" beyond those reductions.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class EsaParams:
    l_I: int
    l_L: int
    k: int
    eps: int
    scale: float = 0.0  # softmax scale; 0 -> 1/sqrt(d)


# ----------------------------------------------------------------------------
# rounding helpers
# ----------------------------------------------------------------------------
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 value (8 significant bits, ties
    to even), returned as float64.  Finite, normal-range inputs."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                      # x = m * 2**e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0), e - 8)


# ----------------------------------------------------------------------------
# Section 3.1: token partition
# ----------------------------------------------------------------------------
def partition(t: int, l_I: int, l_L: int):
    """Preceding tokens [0,t) -> I=[0,i_end), M=[i_end,m_end), L=[m_end,t).
    I and L have fixed lengths and are always kept; M is what lies between."""
    i_end = min(l_I, t)
    m_end = max(i_end, t - l_L)
    return i_end, m_end


# ----------------------------------------------------------------------------
# Eq. 5: linear compression of concatenated heads
# ----------------------------------------------------------------------------
def compress(X: np.ndarray, W: np.ndarray, b=None) -> np.ndarray:
    """X [n, d_in] (heads concatenated), W [d', d_in], optional bias [d'] ->
    bf16-rounded [n, d'].  W is expected already rounded to bf16."""
    Y = np.asarray(X, np.float64) @ np.asarray(W, np.float64).T
    if b is not None:
        Y = Y + np.asarray(b, np.float64)[None, :]
    return bf16_round(Y)


def fold_gqa(W_full: np.ndarray, H: int, H_G: int, d: int) -> np.ndarray:
    """A [d', H*d] key compressor acting on keys whose H_G heads are repeated
    H/H_G times equals a [d', H_G*d] compressor with each group's columns
    summed."""
    dp = W_full.shape[0]
    g = H // H_G
    return np.asarray(W_full, np.float64).reshape(dp, H_G, g, d).sum(axis=2).reshape(dp, H_G * d)


# ----------------------------------------------------------------------------
# Eq. 6, Eq. 4, Eq. 8, Eq. 2
# ----------------------------------------------------------------------------
def scores(qc: np.ndarray, kc_M: np.ndarray) -> np.ndarray:
    """Eq. 6: S[c,m] = q'_c . k'_m  -> fp32 [l_C, l_M]."""
    return (np.asarray(qc, np.float64) @ np.asarray(kc_M, np.float64).T).astype(np.float32)


def aggregate(S: np.ndarray) -> np.ndarray:
    """Eq. 4 in fp32: s_m = max_c ( S[c,m] - max_{m'} S[c,m'] )."""
    S = np.asarray(S, np.float32)
    r = S.max(axis=1, keepdims=True)
    s = (S - r).max(axis=0)
    return s + np.float32(0.0)              # -0 -> +0


def proximity_pool(s: np.ndarray, eps: int) -> np.ndarray:
    """Eq. 8: s'_j = max_{w = max(j-eps, first)}^{min(j+eps, last)} s_w, the
    window clipped to the middle tokens (s covers exactly M)."""
    s = np.asarray(s, np.float32)
    n = s.shape[0]
    out = s.copy()
    for off in range(1, eps + 1):
        if off >= n:
            break
        out[off:] = np.maximum(out[off:], s[:-off])     # neighbour w = j - off
        out[:-off] = np.maximum(out[:-off], s[off:])    # neighbour w = j + off
    return out


def topk(sp: np.ndarray, k: int) -> np.ndarray:
    """Eq. 2: indices (into M) of the k largest scores, larger score first and
    the lower index first among equal scores; returned in ascending order."""
    sp = np.asarray(sp, np.float32)
    k = min(int(k), sp.shape[0])
    order = np.argsort(-sp, kind="stable")
    return np.sort(order[:k]).astype(np.int64)


def select(qc: np.ndarray, kc_M: np.ndarray, k: int, eps: int):
    """Scores -> aggregated -> pooled -> top-k.  Returns (indices into M,
    pooled scores s', row maxima r).  All of M when k >= l_M."""
    l_M = kc_M.shape[0]
    if l_M == 0:
        return np.zeros(0, np.int64), np.zeros(0, np.float32), None
    S = scores(qc, kc_M)
    sp = proximity_pool(aggregate(S), eps)
    if k >= l_M:
        return np.arange(l_M, dtype=np.int64), sp, S.max(axis=1)
    return topk(sp, k), sp, S.max(axis=1)


# ----------------------------------------------------------------------------
# Eq. 3 and Section 4.3: scores without dimensionality reduction
# ----------------------------------------------------------------------------
def scores_full(Q_C: np.ndarray, K_M: np.ndarray) -> np.ndarray:
    """Eq. 3: f_s(m; c) = sum over the H query heads of q_{h,c} . k_{h,m}, where head h reads
    key/value head h // (H/H_G).  Q_C [l_C,H,d], K_M [l_M,H_G,d] -> fp32 [l_C, l_M]."""
    Q_C, K_M = np.asarray(Q_C, np.float64), np.asarray(K_M, np.float64)
    H, g = Q_C.shape[1], Q_C.shape[1] // K_M.shape[1]
    S = np.zeros((Q_C.shape[0], K_M.shape[0]), np.float64)
    for h in range(H):
        S += Q_C[:, h, :] @ K_M[:, h // g, :].T
    return S.astype(np.float32)


def aggregate_per_head(Q_C: np.ndarray, K_M: np.ndarray) -> np.ndarray:
    """Section 4.3, "individual": every head scores the tokens by itself -- Eq. 4 on its own
    logits q_{h,c} . k_{h,m} -- and a token's score is the largest of its H head scores."""
    Q_C, K_M = np.asarray(Q_C, np.float64), np.asarray(K_M, np.float64)
    H, g = Q_C.shape[1], Q_C.shape[1] // K_M.shape[1]
    best = None
    for h in range(H):
        s_h = aggregate((Q_C[:, h, :] @ K_M[:, h // g, :].T).astype(np.float32))
        best = s_h if best is None else np.maximum(best, s_h)
    return best


def select_full(Q_C: np.ndarray, K_M: np.ndarray, k: int, eps: int, per_head: bool = False):
    """Selection on full-dimension scores: Eq. 3 -> Eq. 4 ("uniform", the paper's method without
    compression) or the per-head vote, then Eq. 8 and Eq. 2 as usual.  Returns (indices into M,
    pooled scores)."""
    l_M = K_M.shape[0]
    if l_M == 0:
        return np.zeros(0, np.int64), np.zeros(0, np.float32)
    s = aggregate_per_head(Q_C, K_M) if per_head else aggregate(scores_full(Q_C, K_M))
    sp = proximity_pool(s, eps)
    if k >= l_M:
        return np.arange(l_M, dtype=np.int64), sp
    return topk(sp, k), sp


def recall(sel: np.ndarray, truth: np.ndarray) -> float:
    """Share of the ground-truth selection that another selection also contains (Fig. 3)."""
    truth = np.asarray(truth)
    return float(np.isin(truth, np.asarray(sel)).mean()) if truth.size else 1.0


# ----------------------------------------------------------------------------
# Eq. 1 / Algorithm 1: attention over the reduced key set
# ----------------------------------------------------------------------------
def attend_positions(t: int, l_C: int, sel_abs: np.ndarray, p: EsaParams) -> np.ndarray:
    """Key positions attended by the chunk: I, the selected middle tokens, L,
    then C (C is additionally causal)."""
    i_end, m_end = partition(t, p.l_I, p.l_L)
    return np.concatenate([np.arange(0, i_end), np.asarray(sel_abs, np.int64),
                           np.arange(m_end, t), np.arange(t, t + l_C)]).astype(np.int64)


def attend(Q_C: np.ndarray, K: np.ndarray, V: np.ndarray, sel_abs: np.ndarray, t: int,
           p: EsaParams, return_lse: bool = False, heads=None, Q_global=None, K_global=None):
    """Eq. 1.  Q_C [l_C,H,d]; K,V [>=t+l_C,H_G,d] with C at [t,t+l_C);
    sel_abs absolute positions of the selected middle tokens.  Query head h
    uses key/value head h // (H/H_G).  Query c sees every I, M_k and L key and
    the C keys at chunk offsets <= c (Algorithm 1: non-causal on [I,M_k],
    causal with bottom-right alignment on [L,C]).  Returns float64 [l_C,H,d];
    with ``heads`` given only those query heads are computed (the rest are NaN).

    Section 3.2 (two positions): the logits against I and M_k may use a second
    encoding of the same tokens -- queries ``Q_global`` (all at one fixed
    position) and keys ``K_global`` (all at position 0) -- while the logits
    against L and C use Q_C and K (relative positions).  The softmax still spans
    the union of both sets of logits, which is what Algorithm 1's weighting of
    its two partial results by their normalisers amounts to.  None = the same
    tensors for both parts."""
    Q_C = np.asarray(Q_C, np.float64)
    Qg = Q_C if Q_global is None else np.asarray(Q_global, np.float64)
    Kg = K if K_global is None else K_global
    l_C, H, d = Q_C.shape
    H_G = K.shape[1]
    g = H // H_G
    scale = p.scale if p.scale > 0 else 1.0 / np.sqrt(d)
    pos = attend_positions(t, l_C, sel_abs, p)
    i_far = partition(t, p.l_I, p.l_L)[0] + len(sel_abs)   # |I| + |M_k|
    n_prev = pos.shape[0] - l_C                      # keys before C in the list
    # visible[c, j]: every key before C; C key u visible iff u <= c
    visible = np.ones((l_C, pos.shape[0]), dtype=bool)
    visible[:, n_prev:] = np.tril(np.ones((l_C, l_C), dtype=bool))
    O = np.full((l_C, H, d), np.nan, np.float64)
    LSE = np.full((l_C, H), np.nan, np.float64)
    for h in (range(H) if heads is None else heads):
        Vh = np.asarray(V[pos, h // g, :], np.float64)
        n_far = i_far                                        # list entries of I and M_k come first
        logits = np.concatenate(
            [scale * (Qg[:, h, :] @ np.asarray(Kg[pos[:n_far], h // g, :], np.float64).T),
             scale * (Q_C[:, h, :] @ np.asarray(K[pos[n_far:], h // g, :], np.float64).T)], axis=1)
        logits = np.where(visible, logits, -np.inf)
        mx = logits.max(axis=1, keepdims=True)
        w = np.exp(logits - mx)
        den = w.sum(axis=1, keepdims=True)
        O[:, h, :] = (w / den) @ Vh
        LSE[:, h] = (mx + np.log(den))[:, 0]
    return (O, LSE) if return_lse else O


def softmax_part(Qh, Kh, Vh, scale, mask=None):
    """Attention of the rows of Qh over one set of keys on its own: (normalised output, log of
    the normaliser).  A row that sees no key gives (0, -inf)."""
    logits = scale * (Qh @ Kh.T)
    if mask is not None:
        logits = np.where(mask, logits, -np.inf)
    if logits.shape[1] == 0:
        return np.zeros((Qh.shape[0], Vh.shape[1])), np.full(Qh.shape[0], -np.inf)
    mx = logits.max(axis=1, keepdims=True)
    mx = np.where(np.isfinite(mx), mx, 0.0)
    w = np.exp(logits - mx)
    den = w.sum(axis=1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        out = np.where(den > 0, (w @ Vh) / den, 0.0)
        lse = np.where(den[:, 0] > 0, mx[:, 0] + np.log(den[:, 0]), -np.inf)
    return out, lse


def merge_softmax_parts(parts):
    """Attention over a union of disjoint key sets from the per-set results: each part is
    (normalised output [n, d], log-normaliser [n]); the union's output is the parts' outputs
    weighted by softmax over the parts of their log-normalisers (taken after subtracting the
    largest one).  With two parts this is the weighting step of the paper's Algorithm 1."""
    lse = np.stack([q for _, q in parts], axis=0)               # [parts, n]
    top = lse.max(axis=0, keepdims=True)
    top = np.where(np.isfinite(top), top, 0.0)
    w = np.exp(lse - top)
    w = w / w.sum(axis=0, keepdims=True)
    return sum(wi[:, None] * o for wi, (o, _) in zip(w, parts))


def attend_by_parts(Q_C, K, V, sel_abs, t, p: EsaParams, Q_global=None, K_global=None, cuts=None):
    """The same attention as ``attend`` computed part by part: the key list is cut into pieces
    (by default the two of Algorithm 1: [I, M_k] seen by the far-position queries without a causal
    mask, [L, C] seen by the near-position queries causally), each piece is attended on its own,
    and the pieces are merged by ``merge_softmax_parts``.  ``cuts`` gives other cut points inside
    the key list (any piece lying in the first |I|+|M_k| entries uses the far-position tensors)."""
    Q_C = np.asarray(Q_C, np.float64)
    Qg = Q_C if Q_global is None else np.asarray(Q_global, np.float64)
    Kg = K if K_global is None else K_global
    l_C, H, d = Q_C.shape
    g = H // K.shape[1]
    scale = p.scale if p.scale > 0 else 1.0 / np.sqrt(d)
    pos = attend_positions(t, l_C, sel_abs, p)
    n_far = partition(t, p.l_I, p.l_L)[0] + len(sel_abs)
    n_prev = pos.shape[0] - l_C
    visible = np.ones((l_C, pos.shape[0]), dtype=bool)
    visible[:, n_prev:] = np.tril(np.ones((l_C, l_C), dtype=bool))
    edges = sorted(set([0, n_far, pos.shape[0]] + list(cuts or [])))
    O = np.empty((l_C, H, d), np.float64)
    for h in range(H):
        parts = []
        for a, b in zip(edges[:-1], edges[1:]):
            if a == b:
                continue
            far = b <= n_far
            Qh = (Qg if far else Q_C)[:, h, :]
            Kh = np.asarray((Kg if far else K)[pos[a:b], h // g], np.float64)
            Vh = np.asarray(V[pos[a:b], h // g], np.float64)
            parts.append(softmax_part(Qh, Kh, Vh, scale, visible[:, a:b]))
        O[:, h, :] = merge_softmax_parts(parts)
    return O


# ----------------------------------------------------------------------------
# one whole step
# ----------------------------------------------------------------------------
@dataclass
class StepResult:
    sel_abs: np.ndarray     # ascending absolute positions of M_k
    pooled: np.ndarray      # s' over M (fp32), empty when l_M == 0
    rowmax: np.ndarray      # r_c (fp32) or None
    qc: np.ndarray          # compressed queries (bf16 values as float64)
    O: np.ndarray           # attention output float64 [l_C,H,d]
    O_bf16: np.ndarray      # the same rounded to bf16 values
    i_end: int
    m_end: int


def esa_step(Q_C, K, V, Wq, Wk, p: EsaParams, t: int, bq=None, bk=None, Kc=None,
             do_attend: bool = True, heads=None) -> StepResult:
    """One ESA step on a chunk.  Q_C [l_C,H,d]; K,V [>=t+l_C,H_G,d] (bf16 values);
    Wq [d',d_H], Wk [d',d_G] already rounded to bf16; Kc optionally the cached
    compressed keys [>=t, d'] (else recomputed from K, of which it is a pure
    function)."""
    Q_C = np.asarray(Q_C, np.float64)
    l_C, H, d = Q_C.shape
    i_end, m_end = partition(t, p.l_I, p.l_L)
    qc = compress(Q_C.reshape(l_C, H * d), Wq, bq)
    if m_end > i_end:
        if Kc is None:
            kc_M = compress(np.asarray(K[i_end:m_end], np.float64).reshape(m_end - i_end, -1), Wk, bk)
        else:
            kc_M = np.asarray(Kc[i_end:m_end], np.float64)
        sel, sp, r = select(qc, kc_M, p.k, p.eps)
        sel_abs = sel + i_end
    else:
        sel_abs, sp, r = np.zeros(0, np.int64), np.zeros(0, np.float32), None
    if do_attend:
        O = attend(Q_C, K, V, sel_abs, t, p, heads=heads)
        Ob = bf16_round(O)
    else:
        O = Ob = None
    return StepResult(sel_abs, sp, r, qc, O, Ob, i_end, m_end)


# ----------------------------------------------------------------------------
# Section 3.3 / Appendix A: operation and cache accounting
# ----------------------------------------------------------------------------
def flops_full_attention(d_H, H, l_C, l_total):
    """(4 d_H + 3 H) l_C l_{I,M,L,C}: QK^T, softmax (3 ops per weight), PV."""
    return (4 * d_H + 3 * H) * l_C * l_total


def flops_esa_step(d_H, H, d_c, l_C, l_I, l_M, l_L, k):
    """Appendix A: compression + selection + sparse attention of one step."""
    compression = 2 * 2 * l_C * d_H * d_c + 2 * l_C * d_c
    selection = 2 * l_M * l_C * d_c + l_M * l_C
    sparse = (4 * d_H + 3 * H) * l_C * (l_I + l_L + l_C + k)
    return compression, selection, sparse


def cache_overhead(d_c, d_G):
    """Compressed-key cache relative to the K+V cache: d' / (2 d_G)."""
    return d_c / (2.0 * d_G)
