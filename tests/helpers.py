"""Shared plumbing of the parity tests: seeded inputs -> device tensors, one
step through the C ABI, and the comparison rules.

Comparison rules
  * selected index sets: equal, except that a token may differ when its ORACLE pooled
    score lies within ``band`` of the oracle's k-th score, band = 1e-3 * max(|s'_(k)|,
    max_c |r_c|): the aggregated score is a difference of numbers of size |r_c| and the
    k-th score is often exactly 0, so the relative band is taken against the larger.
  * attention outputs: max-abs <= 2e-2 and mean-abs <= 2e-3 (bf16 output).
  * compressed keys: bit-exact bf16, except that the kernel's value may be the bf16
    rounding of any number within the fp32 accumulation bound of the exact (float64)
    product (the kernel accumulates in fp32, the oracle in float64); at most 0.2 % of
    the elements may differ at all.
"""
from __future__ import annotations

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


def check_index_sets(sel_gpu: np.ndarray, res: "orc.StepResult", k: int, what=""):
    """The band rule above.  Returns the number of differing tokens."""
    sel_or = res.sel_abs
    assert len(sel_gpu) == len(sel_or), f"{what}: count {len(sel_gpu)} != {len(sel_or)}"
    assert np.all(np.diff(sel_gpu) > 0), f"{what}: indices must be ascending and distinct"
    if len(sel_or) == 0:
        return 0
    assert sel_gpu.min() >= res.i_end and sel_gpu.max() < res.m_end, f"{what}: index outside M"
    a, b = set(sel_gpu.tolist()), set(sel_or.tolist())
    if a == b:
        return 0
    sp = res.pooled
    kth = np.sort(sp)[::-1][len(sel_or) - 1]
    band = BAND_REL * max(abs(float(kth)), float(np.max(np.abs(res.rowmax))))
    diff = sorted(a ^ b)
    bad = [m for m in diff if abs(float(sp[m - res.i_end]) - float(kth)) > band]
    assert not bad, (f"{what}: {len(bad)} of {len(diff)} differing tokens lie outside the band "
                     f"{band:.3e} around the k-th score {kth:.6e}; first {bad[:5]}")
    return len(diff)


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
