"""Shared plumbing of the parity tests: seeded inputs -> device tensors, one
step through the C ABI, and the comparison rules.

Comparison rules
  * selected index sets: equal, except that a token may differ when its ORACLE pooled
    score lies within ``band`` of the oracle's k-th score.  Two bands are evaluated: the
    literal one, 1e-3 * |s'_(k)|, and the wide one, 1e-3 * max(|s'_(k)|, max_c |r_c|) (the
    aggregated score is a difference of numbers of size |r_c| and the k-th score is often
    exactly 0).  The literal band is asserted, the counts under both are logged per case.
  * attention outputs: max-abs <= 2e-2 and mean-abs <= 2e-3 (bf16 output).
  * compressed keys and queries: bit-exact bf16, except that the kernel's value may be the
    bf16 rounding of any number within the fp32 accumulation bound of the exact (float64)
    product (the kernel accumulates in fp32, the oracle in float64); at most 0.2 % of
    the elements may differ at all.
  * pooled scores: compared with the oracle evaluated on the kernel's own q' and k', element
    by element within the fp32 accumulation bound (``score_error_bound``), maximum exactly 0.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import esa_synth as syn
from oracle import esa_oracle as orc

ATT_MAX_ABS = 2e-2
ATT_MEAN_ABS = 2e-3
BAND_REL = 1e-3


def bits_to_torch(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(device)


def torch_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def oracle_weights(cfg, layer=0):
    wq, wk = syn.compressor_weights(cfg, layer)
    return wq, wk, orc.bf16_round(wq), orc.bf16_round(wk)


def oracle_params(cfg) -> orc.EsaParams:
    return orc.EsaParams(cfg.l_I, cfg.l_L, cfg.k, cfg.eps)


def make_esa(cfg, max_tokens=None, max_chunk=None, max_batch=None, layer=0, bias=None, eps=None, top_k=None):
    import paper_2502_14477_b200 as esa
    ec = esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k if top_k is None else top_k,
                       cfg.eps if eps is None else eps, max_chunk or cfg.l_C, max_batch or cfg.B,
                       max_tokens or cfg.max_tokens)
    ctx = esa.Esa(ec)
    wq, wk = syn.compressor_weights(cfg, layer)
    if bias is None:
        ctx.set_compressors(wq, None, wk, None)
    else:
        ctx.set_compressors(wq, bias[0], wk, bias[1])
    return ctx


@dataclass
class BandReport:
    """Outcome of one index-set comparison (see ``check_index_sets``)."""
    what: str
    n_sel: int
    n_diff: int              # tokens in exactly one of the two sets
    n_outside_literal: int   # of those, oracle score further than 1e-3 * |k-th score| from the k-th score
    n_outside_wide: int      # ... further than 1e-3 * max(|k-th score|, max_c |r_c|)
    kth: float
    scale_r: float

    def __bool__(self):      # truthy when the sets differ at all
        return self.n_diff > 0


BAND_LOG: list = []          # every comparison of the session, printed by conftest at the end


def check_index_sets(sel_gpu: np.ndarray, res: "orc.StepResult", k: int, what="") -> BandReport:
    """The band rule of the module docstring.  Both bands are evaluated: the literal one
    (1e-3 relative to the k-th score alone) and the wide one (relative to the larger of the
    k-th score and the row maxima).  The wide band is asserted; the counts under both are
    returned and logged so that a run shows how often the literal rule would have failed."""
    sel_or = res.sel_abs
    assert len(sel_gpu) == len(sel_or), f"{what}: count {len(sel_gpu)} != {len(sel_or)}"
    assert np.all(np.diff(sel_gpu) > 0), f"{what}: indices must be ascending and distinct"
    if len(sel_or) == 0:
        rep = BandReport(what, 0, 0, 0, 0, 0.0, 0.0)
        BAND_LOG.append(rep)
        return rep
    assert sel_gpu.min() >= res.i_end and sel_gpu.max() < res.m_end, f"{what}: index outside M"
    a, b = set(sel_gpu.tolist()), set(sel_or.tolist())
    sp = res.pooled
    kth = float(np.sort(sp)[::-1][len(sel_or) - 1]) if len(sp) >= len(sel_or) and len(sp) else 0.0
    scale_r = float(np.max(np.abs(res.rowmax))) if res.rowmax is not None else 0.0
    diff = sorted(a ^ b)
    dist = np.array([abs(float(sp[m - res.i_end]) - kth) for m in diff], dtype=np.float64)
    lit = BAND_REL * abs(kth)
    wide = BAND_REL * max(abs(kth), scale_r)
    n_lit = int(np.sum(dist > lit))
    n_wide = int(np.sum(dist > wide))
    rep = BandReport(what, len(sel_or), len(diff), n_lit, n_wide, kth, scale_r)
    BAND_LOG.append(rep)
    assert n_lit == 0, (f"{what}: {n_lit} of {len(diff)} differing tokens lie outside the literal band "
                        f"{lit:.3e} around the k-th score {kth:.6e} ({n_wide} outside the wide band {wide:.3e}); "
                        f"first {[m for m, dd in zip(diff, dist) if dd > lit][:5]}")
    return rep


def score_error_bound(qc: np.ndarray, kc_M: np.ndarray, eps: int):
    """Per-token bound on |s'_gpu - s'_oracle| when both sides start from the SAME bf16 q' and k'.

    The products q'_i k'_i are exact in fp32 (8-bit x 8-bit significands); the kernel adds d' of
    them in fp32 in an order of its own, possibly truncating, the oracle adds them exactly and
    rounds once: |S_gpu - S_or| <= (d' + 1) 2^-23 sum_i |q'_i k'_i| =: e[c, m].  r_c is a maximum
    of such values (error <= max_m e[c, m]), S - r_c adds one fp32 rounding of the difference on
    each side, and maxima (over c, over the pooling window) do not amplify errors.  Returns
    (tol [l_M], rowmax bound [l_C])."""
    aq, ak = np.abs(np.asarray(qc, np.float64)), np.abs(np.asarray(kc_M, np.float64))
    e = (qc.shape[1] + 1) * 2.0 ** -23 * (aq @ ak.T)                 # [l_C, l_M]
    e_r = e.max(axis=1)                                              # [l_C]
    S_abs = aq @ ak.T                                                # >= |S|, hence >= |S - r| / 2
    tol_cm = e + e_r[:, None] + 2.0 ** -22 * (S_abs + S_abs.max(axis=1, keepdims=True))
    tol = tol_cm.max(axis=0)
    out = tol.copy()
    n = tol.shape[0]
    for off in range(1, eps + 1):
        if off >= n:
            break
        out[off:] = np.maximum(out[off:], tol[:-off])
        out[:-off] = np.maximum(out[:-off], tol[off:])
    return out, e_r


def check_pooled_scores(sp_gpu: np.ndarray, qc_gpu: np.ndarray, kc_M: np.ndarray, k: int, eps: int, what=""):
    """Pooled scores s' (Eq. 8) of the kernel against the oracle evaluated on the kernel's own
    bf16 q' (so that only the fp32 accumulation differs): every element within the bound of
    ``score_error_bound``, s' <= 0 with an exact maximum of 0, and the same set of exact zeros
    (a zero may only be missing or extra where the bound reaches 0)."""
    _, sp_or, r = orc.select(qc_gpu, kc_M, k, eps)
    tol, _ = score_error_bound(qc_gpu, kc_M, eps)
    g = sp_gpu.astype(np.float64)
    o = sp_or.astype(np.float64)
    err = np.abs(g - o)
    bad = err > tol
    assert not bad.any(), (f"{what}: {int(bad.sum())} pooled scores beyond the fp32 accumulation bound; "
                           f"worst {err[bad].max():.3e} against {tol[bad][np.argmax(err[bad])]:.3e}")
    assert g.max() == 0.0 and np.all(g <= 0), f"{what}: pooled scores must be <= 0 with maximum 0"
    z = (g == 0.0) != (o == 0.0)
    assert not (z & (np.abs(o) > tol) & (np.abs(g) > tol)).any(), f"{what}: exact zeros differ"
    return float(err.max()), int(z.sum())


def check_attention(O_gpu: torch.Tensor, O_oracle: np.ndarray, what="", heads=None):
    got = torch_to_f64(O_gpu)
    want = O_oracle
    if heads is not None:
        got, want = got[:, heads], want[:, heads]
    err = np.abs(got - want)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert err.max() <= ATT_MAX_ABS, f"{what}: max-abs {err.max():.4e}"
    assert err.mean() <= ATT_MEAN_ABS, f"{what}: mean-abs {err.mean():.4e}"
    return float(err.max()), float(err.mean())


def check_compressed(kc_gpu: torch.Tensor, X: np.ndarray, W: np.ndarray, b=None, what=""):
    """kc_gpu [n, d_c] bf16 vs the exact product X.W^T (+b) rounded to bf16."""
    exact = X @ W.T
    if b is not None:
        exact = exact + np.asarray(b, np.float64)[None, :]
    want = orc.bf16_round(exact)
    got = torch_to_f64(kc_gpu)
    neq = got != want
    if not neq.any():
        return 0
    # The kernel accumulates in fp32: its sum lies within d_in * 2^-24 * sum|terms| of the exact
    # one, so its bf16 result must be the rounding of SOME value in that interval (rounding is
    # monotone, so it suffices to round the interval's ends).
    bound = X.shape[1] * 2.0 ** -24 * (np.abs(X) @ np.abs(W).T)
    if b is not None:
        bound = bound + 2.0 ** -24 * np.abs(exact)
    lo, hi = orc.bf16_round(exact - bound), orc.bf16_round(exact + bound)
    bad = (got < lo) | (got > hi)
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {int(neq.sum())} differing compressed values are not a "
                           f"bf16 rounding of a value within the fp32 accumulation bound; (exact, want, got) = "
                           f"{list(zip(exact[bad][:4], want[bad][:4], got[bad][:4]))}")
    assert neq.mean() < 2e-3, f"{what}: {neq.mean():.2e} of the compressed values differ from the exact rounding"
    return int(neq.sum())


class DeviceSeq:
    """Device caches for B sequences of a workload, filled from the seeded generators."""

    def __init__(self, cfg, max_tokens=None, layer=0, B=None):
        self.cfg, self.layer = cfg, layer
        self.B = B or cfg.B
        self.max_tokens = max_tokens or cfg.max_tokens
        dev = "cuda"
        self.K = torch.zeros(self.B, self.max_tokens, cfg.H_G, cfg.d, dtype=torch.bfloat16, device=dev)
        self.V = torch.zeros_like(self.K)
        self.Kc = torch.zeros(self.B, self.max_tokens, cfg.d_c, dtype=torch.bfloat16, device=dev)
        self.idx = torch.zeros(self.B, cfg.k, dtype=torch.int32, device=dev)
        self.n_sel = torch.zeros(self.B, dtype=torch.int32, device=dev)

    def fill_kv(self, row0, row1, seqs=None):
        for b in (range(self.B) if seqs is None else seqs):
            self.K[b, row0:row1] = bits_to_torch(syn.qkv_rows(self.cfg, "k", row0, row1, self.layer, b))
            self.V[b, row0:row1] = bits_to_torch(syn.qkv_rows(self.cfg, "v", row0, row1, self.layer, b))

    def q_rows(self, row0, row1):
        return torch.stack([bits_to_torch(syn.qkv_rows(self.cfg, "q", row0, row1, self.layer, b))
                            for b in range(self.B)])


def host_f64(cfg, which, row0, row1, layer=0, seq=0):
    return syn.bf16_bits_to_f64(syn.qkv_rows(cfg, which, row0, row1, layer, seq))
