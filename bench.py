#!/usr/bin/env python
"""Benchmark of the ESA select-plus-attend step on B200.

Headline workload (config "c5" shape): one layer of the Llama-3-8B attention
shape (H=32, H_G=8, d=128, d'=128), a 131072-token chunked prefill in chunks of
512 with l_I=128, l_L=2048, k=4096, eps=3, mixture keys with planted needle
spans.  One bench "step" is the whole chunked prefill of one layer: 256 ESA steps,
each = esa_compress_keys + esa_select + esa_attend.  The metric is prefill
tokens/s through the 32-layer stack (= 131072 / (32 x layer time)); the layers
are independent and identically shaped, and the timed steps cycle over
``--layers`` distinct layers' data.  The decode workload ("c3": 8 sequences x
131072 cached tokens, one query each, 256 steps) is timed in the same run and
reported under "decode".

Launch: ``python bench.py --gpus N --steps K --warmup W``; for N > 1 under
torchrun, one rank per GPU, every rank an independent replica of the workload
(the step has no cross-GPU exchange), value = total tokens / max-over-ranks time.
``--impl reference`` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import esa_synth as syn

N_LAYERS_STACK = 32
# dram__bytes_read.sum + dram__bytes_write.sum from the ncu captures summarised in
# profiles/dram_bytes_per_kernel.txt (same kernels, same launch shapes as the timed workloads).
ATTEND_TC_DRAM_BYTES = 32087552 + 1280
DECODE_STEP_DRAM_BYTES = (205836544 + 79360) + 39168 + 300288 + 1133312 + (264913408 + 626688) + 4355328


# ----------------------------------------------------------------------------
# small helpers (also exercised by the CPU tests)
# ----------------------------------------------------------------------------
def shard_units(total: int, rank: int, world: int):
    """Contiguous share [lo, hi) of ``total`` independent units for ``rank``."""
    base, rem = divmod(total, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def max_over_ranks(value: float, device=None) -> float:
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "tflops_burst": p["bf16_tflops"],
                "tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


def attend_flops(cfg, t: int, l_C: int) -> float:
    """Algorithmic flops of one esa_attend launch: 4 d_H l_C (n_att - l_C/2)."""
    i_end = min(cfg.l_I, t)
    m_end = max(i_end, t - cfg.l_L)
    n_att = i_end + min(cfg.k, m_end - i_end) + (t - m_end) + l_C
    return 4.0 * cfg.d_H * l_C * (n_att - l_C / 2.0)


def score_flops(cfg, t: int, l_C: int) -> float:
    """One scoring pass (the method's own count): 2 l_C l_M d' + l_C l_M."""
    i_end = min(cfg.l_I, t)
    l_M = max(i_end, t - cfg.l_L) - i_end
    return (2.0 * cfg.d_c + 1.0) * l_C * l_M if l_M > cfg.k else 0.0


def partition_sizes(cfg, t: int, l_C: int):
    i_end = min(cfg.l_I, t)
    m_end = max(i_end, t - cfg.l_L)
    l_M = m_end - i_end
    return i_end, l_M, i_end + min(cfg.k, l_M) + (t - m_end) + l_C


def compress_flops(cfg, l_C: int) -> float:
    """Eq. 5 for the chunk's keys and queries: 2 l_C d' (d_H + d_G)."""
    return 2.0 * l_C * cfg.d_c * (cfg.d_H + cfg.d_G)


def select_bytes(cfg, t: int, l_C: int) -> float:
    """Eq. 2: read 4 l_M, write 4 k (only when l_M > k)."""
    _, l_M, _ = partition_sizes(cfg, t, l_C)
    return 4.0 * l_M + 4.0 * cfg.k if l_M > cfg.k else 0.0


def kernel_rooflines(prof: dict, sampled, cfg, peaks):
    """Per-kernel achieved rates of the profiled chunks: algorithmic work of those chunks / summed
    CUDA-event time of the kernel class, against the measured sustained and burst bf16 peaks
    (contractions) or the measured copy bandwidth (selection)."""
    sc = sum(score_flops(cfg, t, l_C) for t, l_C in sampled)
    out = {}

    def tensor(name, flops, note=None):
        if name not in prof or prof[name][1] <= 0:
            return
        n, ms = prof[name]
        tf = flops / (ms * 1e-3) / 1e12
        out[name] = {"bound": "tensor", "launches": n, "us_per_launch": 1e3 * ms / n, "achieved": tf, "unit": "TFLOP/s",
                     "frac_sustained": tf / peaks["tflops_sustained"], "frac_burst": tf / peaks["tflops_burst"]}
        if note:
            out[name]["note"] = note

    tensor("attend_tc_kernel", sum(attend_flops(cfg, t, l_C) for t, l_C in sampled))
    tensor("score_tc_kernel<.,1>", sc, "one pass: (2 d' + 1) l_C l_M flops per launch")
    tensor("score_tc_kernel<.,2>", sc, "second pass over the same products (the method counts one), with Eq. 4, Eq. 8 and the first radix digit in the epilogue")
    tensor("compress_tc_kernel", sum(compress_flops(cfg, l_C) for t, l_C in sampled),
           "both compressions of a chunk (keys on the side stream, queries ahead of the scoring); latency-bound launches")
    if "score_tc_kernel<.,1>" in out and "score_tc_kernel<.,2>" in out:
        ms = prof["score_tc_kernel<.,1>"][1] + prof["score_tc_kernel<.,2>"][1]
        tf = sc / (ms * 1e-3) / 1e12
        out["scoring, both passes against the method's one-pass work"] = {
            "bound": "tensor", "achieved": tf, "unit": "TFLOP/s", "frac_sustained": tf / peaks["tflops_sustained"],
            "frac_burst": tf / peaks["tflops_burst"]}
    if "select_topk_kernel" in prof and prof["select_topk_kernel"][1] > 0:
        n, ms = prof["select_topk_kernel"]
        gbs = sum(select_bytes(cfg, t, l_C) for t, l_C in sampled) / (ms * 1e-3) / 1e9
        out["select_topk_kernel"] = {"bound": "latency", "launches": n, "us_per_launch": 1e3 * ms / n, "achieved": gbs,
                                     "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                     "note": "read 4 l_M + write 4 k bytes per launch: far too little to load HBM"}
    return out


def decode_bytes(cfg, t: int) -> float:
    """Algorithmic HBM bytes of one decode step of one sequence: 2 l_M d' + 4 n_att d_G."""
    i_end = min(cfg.l_I, t)
    m_end = max(i_end, t - cfg.l_L)
    l_M = m_end - i_end
    n_att = i_end + min(cfg.k, l_M) + (t - m_end) + 1
    return 2.0 * l_M * cfg.d_c + 4.0 * n_att * cfg.d_G


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# workloads on the device
# ----------------------------------------------------------------------------
def bits_to_dev(bits, pin=False):
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    return t.pin_memory() if pin else t.cuda()


class PrefillLayer:
    """One layer of a prefill workload: Q/K/V resident in HBM, caches sized for S tokens."""

    def __init__(self, cfg, layer, keep_host=False):
        S = cfg.S
        self.cfg = cfg
        qb = syn.qkv_rows(cfg, "q", 0, S, layer)
        kb = syn.qkv_rows(cfg, "k", 0, S, layer)
        vb = syn.qkv_rows(cfg, "v", 0, S, layer)
        self.Q = bits_to_dev(qb)[None]          # [1,S,H,d]
        self.K = bits_to_dev(kb)[None]          # [1,S,H_G,d]  (the K cache; C's rows are in place)
        self.V = bits_to_dev(vb)[None]
        self.host = None
        if keep_host:
            self.host = tuple(bits_to_dev(x, pin=True) for x in (qb, kb, vb))
        self.wq, self.wk = syn.compressor_weights(cfg, layer)


def make_ctx(cfg, max_tokens, max_chunk, max_batch):
    import paper_2502_14477_b200 as esa
    return esa.Esa(esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps,
                                 max_chunk, max_batch, max_tokens))


_SIDE = []


def _side_stream():
    if not _SIDE:
        _SIDE.append(torch.cuda.Stream())
    return _SIDE[0]


PROFILE_EVERY = 32     # one chunk in this many runs with per-kernel CUDA events (see run_prefill_layer)


def run_prefill_layer(ctx, cfg, L, bufs, sampled=None, phase=0):
    """The whole chunked prefill of one layer with inputs resident in HBM.

    sampled: list that receives (t, l_C) of the chunks whose kernels were individually timed.  On
    such a chunk the library brackets every kernel with CUDA events on the launching stream
    (esa_set_profiling).  An event record between two kernels keeps the second one from starting
    under the first one (programmatic dependent launch; the attention kernel reads the older rows
    beside the selection kernel), which costs a sampled chunk about a quarter of its time: measured
    163k / 169k / 172k tokens/s with one chunk in 8 / 16 / 32 sampled.  So one chunk in
    PROFILE_EVERY is, the sampled positions moving with `phase` (step number)."""
    Kc, idx, n_sel, O = bufs
    # The compressed keys of the current chunk are not read by this chunk's selection (C is not
    # part of M): esa_compress_keys runs on a side stream beside the attention, and the selection
    # waits for the previous chunk's compression, which covers every row that M can contain.
    main = torch.cuda.current_stream()
    side = _side_stream()
    side.wait_stream(main)
    done = []                                   # done[c]: rows of chunk c are compressed
    for t in range(0, cfg.S, cfg.l_C):
        l_C = min(cfg.l_C, cfg.S - t)
        Qc = L.Q[:, t: t + l_C]
        timed = sampled is not None and (t // cfg.l_C + 5 * phase) % PROFILE_EVERY == 0
        if timed:
            ctx.set_profiling(True)
        with torch.cuda.stream(side):
            ctx.compress_keys(L.K[:, t: t + l_C], Kc, [t])
            ev = torch.cuda.Event()
            ev.record(side)
            done.append(ev)
        # M = [i_end, m_end): the last chunk that reaches into it.  It was enqueued l_L tokens ago and has
        # normally finished: then no wait is put between the attention and the next selection (a stream
        # wait would keep the selection's first kernel from being set up under the attention's tail).
        m_end = max(min(cfg.l_I, t), t - cfg.l_L)
        c_need = (m_end + cfg.l_C - 1) // cfg.l_C - 1
        if c_need >= 0 and not done[c_need].query():
            main.wait_event(done[c_need])
        ctx.select(Qc, Kc, [t], idx, n_sel)
        ctx.attend(Qc, L.K, L.V, [t], idx, n_sel, O[:, t: t + l_C])
        if timed:
            ctx.set_profiling(False)
            sampled.append((t, l_C))
    main.wait_stream(side)


E2E_GROUP = 8          # chunks per host<->device transfer of the end-to-end leg


def run_prefill_layer_e2e(ctx, cfg, L, bufs, caches, stage, O_host, streams):
    """Same work with HOST inputs and outputs: the Q/K/V rows of every chunk are copied from pinned host
    memory, the K/V rows appended to the device caches by esa_append_kv, and O is copied back to host
    memory.  The copies run on their own streams through two sets of staging buffers of E2E_GROUP chunks
    each, so the transfer of group g+1 and the read-back of group g-1 overlap the kernels of group g; the
    library calls are enqueued chunk by chunk on the compute stream (the caller's stream, as any user
    would).  (One transfer per chunk left the leg bound by the host: 180 us of Python per chunk for 13
    stream operations, against 94 us of kernels and 120 us of PCIe time.  Measured with 1 / 2 / 4 / 8 / 16
    chunks per transfer: 90k / 103k / 113k / 117k / 117k tokens/s; at 8 the host-to-device copies run at
    46 GB/s, the leg is bound by PCIe.)"""
    Kc, idx, n_sel, _ = bufs
    Kcache, Vcache = caches
    hq, hk, hv = L.host
    s_in, s_cmp, s_out = streams
    cur = torch.cuda.current_stream()
    for s in streams:
        s.wait_stream(cur)
    in_done = [torch.cuda.Event() for _ in range(2)]
    cmp_done = [torch.cuda.Event() for _ in range(2)]
    out_done = [torch.cuda.Event() for _ in range(2)]
    rows = E2E_GROUP * cfg.l_C
    for g, t0 in enumerate(range(0, cfg.S, rows)):
        n = min(rows, cfg.S - t0)
        slot = g & 1
        Qs, Ks, Vs, Os = stage[slot]
        with torch.cuda.stream(s_in):
            if g >= 2:
                s_in.wait_event(cmp_done[slot])          # the kernels of group g-2 have read this slot
            Qs[0, :n].copy_(hq[t0: t0 + n], non_blocking=True)
            Ks[0, :n].copy_(hk[t0: t0 + n], non_blocking=True)
            Vs[0, :n].copy_(hv[t0: t0 + n], non_blocking=True)
            in_done[slot].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(in_done[slot])
            if g >= 2:
                s_cmp.wait_event(out_done[slot])         # group g-2's output has left this slot
            for o in range(0, n, cfg.l_C):
                t, l_C = t0 + o, min(cfg.l_C, n - o)
                ctx.append_kv(Ks[:, o: o + l_C], Vs[:, o: o + l_C], Kcache, Vcache, [t])
                ctx.compress_keys(Ks[:, o: o + l_C], Kc, [t])
                ctx.select(Qs[:, o: o + l_C], Kc, [t], idx, n_sel)
                ctx.attend(Qs[:, o: o + l_C], Kcache, Vcache, [t], idx, n_sel, Os[:, o: o + l_C])
            cmp_done[slot].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(cmp_done[slot])
            O_host[t0: t0 + n].copy_(Os[0, :n], non_blocking=True)
            out_done[slot].record(s_out)
    for s in streams:
        cur.wait_stream(s)


# ----------------------------------------------------------------------------
# the two arms
# ----------------------------------------------------------------------------
def oracle_sample(cfg, layer, chunks, heads=None):
    """Times the CPU oracle on a few chunks of the prefill workload; returns
    (tokens processed, seconds, description)."""
    from oracle import esa_oracle as orc
    wq, wk = syn.compressor_weights(cfg, layer)
    Wq, Wk = orc.bf16_round(wq), orc.bf16_round(wk)
    p = orc.EsaParams(cfg.l_I, cfg.l_L, cfg.k, cfg.eps)
    t_max = max(chunks) * cfg.l_C + cfg.l_C
    K = syn.bf16_bits_to_f64(syn.qkv_rows(cfg, "k", 0, t_max, layer))
    V = syn.bf16_bits_to_f64(syn.qkv_rows(cfg, "v", 0, t_max, layer))
    Kc = orc.compress(K.reshape(t_max, -1), Wk)          # the cache carried between steps
    secs, toks = 0.0, 0
    for c in chunks:
        t = c * cfg.l_C
        Q = syn.bf16_bits_to_f64(syn.qkv_rows(cfg, "q", t, t + cfg.l_C, layer))
        t0 = time.perf_counter()
        orc.esa_step(Q, K[: t + cfg.l_C], V[: t + cfg.l_C], Wq, Wk, p, t, Kc=Kc, heads=heads)
        secs += time.perf_counter() - t0
        toks += cfg.l_C
    return toks, secs, f"chunks {list(chunks)} of layer {layer} (all heads), k' cache precomputed"


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    chunks = [13, 255]                       # first chunk with l_M > k, and the last
    total = args.steps + args.warmup
    secs_all = []
    for s in range(total):
        toks, secs, what = oracle_sample(cfg, s % 2, chunks)
        if s >= args.warmup:
            secs_all.append(secs / toks)
    per_tok = sum(secs_all) / len(secs_all)
    value = 1.0 / (per_tok * N_LAYERS_STACK)
    line = {
        "impl": "reference", "metric": "esa_prefill_tokens_per_s_128k", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * per_tok * len(chunks) * cfg.l_C, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                         "sample": f"each step: {what}; per-token time extrapolated to the 32-layer stack"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(cfg):
    return {"workload": "c5: Llama-3-8B attention shape, 131072-token prefill in chunks of 512, "
                        "l_I=128 l_L=2048 k=4096 eps=3 d'=128, mixture keys + planted needles; "
                        "a step = one layer's whole chunked prefill, value = tokens/s through 32 such layers",
            "H": cfg.H, "H_G": cfg.H_G, "head_dim": cfg.d, "d_c": cfg.d_c, "l_C": cfg.l_C, "S": cfg.S,
            "l2": "per-layer inputs (1.6 GB) exceed the 126 MB L2; steps cycle over distinct layers"}


def time_decode(cfg3, n_steps, rank_seed):
    """Config c3: B sequences with S cached tokens, n_steps decode steps (append K/V,
    compress the new key, select, attend).  Returns (us/step, bytes/step, launches/step)."""
    B, S = cfg3.B, cfg3.S
    n = S + n_steps
    ctx = make_ctx(cfg3, n, 1, B)
    wq, wk = syn.compressor_weights(cfg3)
    ctx.set_compressors(wq, None, wk, None)
    g = torch.Generator(device="cuda")
    g.manual_seed(cfg3.seed + 1000 * rank_seed)
    # decode inputs are N(0,1) bf16; drawn on the device (2 x 2.2 GB) to keep start-up short
    K = torch.randn(B, n, cfg3.H_G, cfg3.d, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(B, n, cfg3.H_G, cfg3.d, device="cuda", dtype=torch.bfloat16, generator=g)
    Qs = torch.randn(n_steps, B, 1, cfg3.H, cfg3.d, device="cuda", dtype=torch.bfloat16, generator=g)
    Knew = K[:, S:].transpose(0, 1).contiguous().unsqueeze(2)      # [step, B, 1, H_G, d]: one contiguous block per step
    Vnew = V[:, S:].transpose(0, 1).contiguous().unsqueeze(2)
    Kc = torch.zeros(B, n, cfg3.d_c, dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, S, 4096):
        ctx.compress_keys(K[:, r0: r0 + 4096].contiguous(), Kc, [r0] * B)
    idx = torch.zeros(B, cfg3.k, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(B, dtype=torch.int32, device="cuda")
    O = torch.empty(B, 1, cfg3.H, cfg3.d, dtype=torch.bfloat16, device="cuda")

    main = torch.cuda.current_stream()
    side = _side_stream()
    side.wait_stream(main)
    done = {}                                   # done[i]: the compressed key of step i's token is in place

    def step(i):
        # the new token's compressed key is not read by this step's selection (it enters M l_L steps
        # later): side stream, and a wait only for a step whose key is needed and not yet written
        t = [S + i] * B
        kn, vn = Knew[i], Vnew[i]
        with torch.cuda.stream(side):
            ctx.compress_keys(kn, Kc, t)
            ev = torch.cuda.Event()
            ev.record(side)
            done[i] = ev
        ctx.append_kv(kn, vn, K, V, t)
        need = i - cfg3.l_L - 1                 # last step whose token is inside M now
        if need in done and not done[need].query():
            main.wait_event(done[need])
        done.pop(need - 1, None)
        ctx.select(Qs[i], Kc, t, idx, n_sel)
        ctx.attend(Qs[i], K, V, t, idx, n_sel, O)

    for i in range(min(8, n_steps)):
        step(i)
    torch.cuda.synchronize()
    # per-kernel times of a few steps, outside the timed region (events between the kernels of a step
    # keep each from starting under its predecessor's tail)
    ctx.set_profiling(True)
    for i in range(min(8, n_steps)):
        step(i)
    ctx.set_profiling(False)
    torch.cuda.synchronize()
    prof = {k: {"launches": n, "us_per_launch": 1e3 * ms / n} for k, (n, ms) in ctx.read_profile().items()}
    l0 = ctx.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n_steps):
        step(i)
    main.wait_stream(side)
    e1.record()
    torch.cuda.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / n_steps
    byts = B * sum(decode_bytes(cfg3, S + i) for i in range(n_steps)) / n_steps
    launches = (ctx.launch_count - l0) / n_steps
    assert ctx.last_device_status() == 0
    ctx.close()
    return us, byts, launches, prof


class DeviceLayer:
    """Q/K/V of one layer drawn on the device (N(0,1) bf16, optional per-head scale U(0.5, 2)): the
    secondary prefill legs use it to keep start-up short."""

    def __init__(self, cfg, seed):
        g = torch.Generator(device="cuda")
        g.manual_seed(seed)
        mk = lambda nh: torch.randn(1, cfg.S, nh, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
        self.Q, self.K, self.V = mk(cfg.H), mk(cfg.H_G), mk(cfg.H_G)
        if cfg.kind == "headscale":
            for x in (self.Q, self.K, self.V):
                x.mul_((0.5 + 1.5 * torch.rand(1, 1, x.shape[2], 1, device="cuda", generator=g)).to(torch.bfloat16))
        self.wq, self.wk = syn.compressor_weights(cfg, 0)


def time_prefill_leg(name, steps, peaks):
    """Whole chunked prefill of one layer of a secondary workload (c2: 32k, c4: 256k in chunks of 1024)."""
    cfg = syn.get_config(name)
    L = DeviceLayer(cfg, cfg.seed)
    ctx = make_ctx(cfg, cfg.S, cfg.l_C, 1)
    ctx.set_compressors(L.wq, None, L.wk, None)
    bufs = (torch.zeros(1, cfg.S, cfg.d_c, dtype=torch.bfloat16, device="cuda"),
            torch.zeros(1, cfg.k, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"),
            torch.empty(1, cfg.S, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda"))
    for i in range(2):
        run_prefill_layer(ctx, cfg, L, bufs)
    torch.cuda.synchronize()
    ctx.read_profile()
    sampled = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        run_prefill_layer(ctx, cfg, L, bufs, sampled, phase=i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert ctx.last_device_status() == 0
    prof = ctx.read_profile()
    by_kernel = kernel_rooflines(prof, sampled, cfg, peaks)
    n_chunks = (cfg.S + cfg.l_C - 1) // cfg.l_C
    att_ms = sum(v[1] for k, v in prof.items() if k.startswith("attend"))
    out = {"workload": f"{name}: H={cfg.H} H_G={cfg.H_G} d={cfg.d} d'={cfg.d_c}, {cfg.S}-token prefill in chunks of {cfg.l_C}, "
                       f"l_I={cfg.l_I} l_L={cfg.l_L} k={cfg.k} eps={cfg.eps}; inputs drawn on the device",
           "ms_per_layer": ms, "tokens_per_s_per_layer": cfg.S / (ms * 1e-3), "steps": steps,
           "attention_share_of_step": att_ms * (steps * n_chunks / max(1, len(sampled))) / (ms * steps),
           "roofline_by_kernel": by_kernel}
    ctx.close()
    del L, bufs
    torch.cuda.empty_cache()
    return out


def time_extensions(peaks):
    """The steps next to the measured path, each on the c5 shape (512 queries after 65536 cached tokens unless
    noted), timed with the library's per-kernel CUDA events over a few repetitions: two-position attention
    (Section 3.2), full-dimension and per-head selection (Eq. 3, Section 4.3), attention with the K/V cache
    in host memory (appendix "Model Loading") and compressor fitting (Eq. 7)."""
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config("c5")
    t, l_C, reps = 65536, cfg.l_C, 5
    n = t + l_C
    ctx = make_ctx(cfg, n, l_C, 1)
    wq, wk = syn.compressor_weights(cfg)
    ctx.set_compressors(wq, None, wk, None)
    g = torch.Generator(device="cuda").manual_seed(11)
    mk = lambda *shape: torch.randn(*shape, device="cuda", dtype=torch.bfloat16, generator=g)
    K, V, Kf = mk(1, n, cfg.H_G, cfg.d), mk(1, n, cfg.H_G, cfg.d), mk(1, n, cfg.H_G, cfg.d)
    Q, Qf = mk(1, l_C, cfg.H, cfg.d), mk(1, l_C, cfg.H, cfg.d)
    idx = torch.zeros(1, cfg.k, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(1, dtype=torch.int32, device="cuda")
    O = torch.empty_like(Q)
    i_end, l_M, n_att = partition_sizes(cfg, t, l_C)
    idx[0] = (torch.sort(torch.randperm(l_M, device="cuda", generator=g)[: cfg.k])[0] + i_end).to(torch.int32)
    n_sel[0] = cfg.k
    out = {"shape": f"c5 shape, {l_C} queries after {t} cached tokens, {reps} repetitions each, inputs drawn on the device"}

    def timed(fn, name):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ctx.read_profile()
        ctx.set_profiling(True)
        for _ in range(reps):
            fn()
        ctx.set_profiling(False)
        torch.cuda.synchronize()
        return {k: 1e3 * ms / cnt for k, (cnt, ms) in ctx.read_profile().items()}

    fl_att = attend_flops(cfg, t, l_C)
    one = timed(lambda: ctx.attend(Q, K, V, [t], idx, n_sel, O), "attend")["attend_tc_kernel"]
    two = timed(lambda: ctx.attend_two_position(Q, Qf, K, Kf, V, [t], idx, n_sel, O), "attend2")["attend_tc_kernel"]
    out["two_position_attention"] = {"us_per_launch": two, "one_position_us_per_launch": one,
                                     "achieved_tflops": fl_att / two * 1e-6, "frac_burst": fl_att / two * 1e-6 / peaks["tflops_burst"]}
    fl_full = 2.0 * 2.0 * cfg.d_H * l_C * l_M          # two passes over all heads and dimensions
    for per_head, key in ((False, "select_full_uniform"), (True, "select_full_per_head")):
        pr = timed(lambda: ctx.select_full(Q, K, [t], idx, n_sel, per_head=per_head), key)
        us = pr["score_full_kernel<.,1>+<.,2>"]
        out[key] = {"score_us_per_call": us, "achieved_tflops": fl_full / us * 1e-6, "frac_burst": fl_full / us * 1e-6 / peaks["tflops_burst"],
                    "pool_hist_us": pr.get("pool_hist_kernel"), "select_topk_us": pr.get("select_topk_kernel"),
                    "note": "mma.sync kernels (both passes timed together); flops = 2 passes x 2 d_H l_C l_M"}
    idx[0] = (torch.sort(torch.randperm(l_M, device="cuda", generator=g)[: cfg.k])[0] + i_end).to(torch.int32)
    n_sel[0] = cfg.k
    K_host, V_host = K.cpu().pin_memory(), V.cpu().pin_memory()
    stage_rows = cfg.l_I + cfg.k + cfg.l_L + l_C
    Ks = torch.empty(1, stage_rows, cfg.H_G, cfg.d, dtype=torch.bfloat16, device="cuda")
    Vs = torch.empty_like(Ks)
    pr = timed(lambda: ctx.attend_host_kv(Q, K_host, V_host, [t], idx, n_sel, Ks, Vs, O), "host")
    gbytes = 2.0 * n_att * cfg.d_G * 2
    out["host_resident_kv"] = {"gather_us": pr["gather_kv_kernel"], "attend_us": pr["attend_tc_kernel"],
                               "gathered_bytes": gbytes, "host_to_device_gbs": gbytes / pr["gather_kv_kernel"] * 1e-3,
                               "note": "rows of I, M_k, L, C read from pinned host memory by the gather kernel (PCIe-bound)"}
    ctx.close()
    # Eq. 7: fitting steps at the Llama shape, batches of 128 pairs
    nb, steps = 128, 60
    fit = esa.EsaFit(esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps, 1, 1, 16), nb, 5e-4)
    fit.set_weights(wq, None, wk, None)
    Qb, Kb = mk(nb, cfg.H, cfg.d), mk(nb, cfg.H_G, cfg.d)
    for _ in range(5):
        fit.step(Qb, Kb)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fit.step(Qb, Kb)
    e1.record()
    torch.cuda.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / steps
    fl = 4.0 * nb * cfg.d_c * (cfg.d_H + cfg.d_G) + 2.0 * nb * nb * (cfg.d_G + 3 * cfg.d_c)
    out["compressor_fitting"] = {"us_per_step": us, "steps_per_s": 1e6 / us, "achieved_tflops_fp32": fl / us * 1e-6,
                                 "launches_per_step": fit.launch_count / (steps + 5), "bound": "launch latency / fp32 ALU",
                                 "note": "batch of 128 pairs, fp32 kernels; the paper's 10 epochs over 50k pairs are 3900 such steps"}
    fit.close()
    del K, V, Kf, K_host, V_host
    torch.cuda.empty_cache()
    return out


def profile_case(args):
    """Small, self-ending cases for ncu captures: every kernel of one ESA step, ``--reps`` times, on
    inputs larger than L2 but well under a few GB.  Inputs are N(0,1) bf16 drawn on the device."""
    import paper_2502_14477_b200 as esa
    H, HG, d, dc = 32, 8, 128, 128
    g = torch.Generator(device="cuda").manual_seed(0)
    wq = (torch.randn(dc, H * d, generator=torch.Generator().manual_seed(1)) / (H * d) ** 0.5).numpy()
    wk = (torch.randn(dc, HG * d, generator=torch.Generator().manual_seed(2)) / (HG * d) ** 0.5).numpy()
    if args.profile_case == "prefill":
        l_C, t, B = 512, args.profile_t, 1
        n = t + l_C
    else:
        l_C, t, B = 1, args.profile_t, 8
        n = t + args.reps + 1
    ctx = esa.Esa(esa.EsaConfig(H, HG, d, dc, 128, 2048, 4096, 3, l_C, B, n))
    ctx.set_compressors(wq, None, wk, None)
    K = torch.randn(B, n, HG, d, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(B, n, HG, d, device="cuda", dtype=torch.bfloat16, generator=g)
    Q = torch.randn(B, l_C, H, d, device="cuda", dtype=torch.bfloat16, generator=g)
    Kc = torch.zeros(B, n, dc, dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, t, 4096):
        r1 = min(t, r0 + 4096)
        ctx.compress_keys(K[:, r0:r1].contiguous(), Kc, [r0] * B)
    idx = torch.zeros(B, 4096, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(B, dtype=torch.int32, device="cuda")
    O = torch.empty_like(Q)
    torch.cuda.synchronize()
    ctx.set_profiling(True)
    for i in range(args.reps):
        tt = [t + (i if l_C == 1 else 0)] * B
        ctx.compress_keys(K[:, tt[0]: tt[0] + l_C].contiguous(), Kc, tt)
        ctx.select(Q, Kc, tt, idx, n_sel)
        ctx.attend(Q, K, V, tt, idx, n_sel, O)
    ctx.set_profiling(False)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    prof = {k: {"launches": n_, "us_per_launch": round(1e3 * ms / n_, 2)} for k, (n_, ms) in ctx.read_profile().items()}
    print(json.dumps({"profile_case": args.profile_case, "t": t, "reps": args.reps, "launches": ctx.launch_count,
                      "kernels_isolated": prof}))


def run_esa(args, cfg):
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()

    n_res = max(1, min(args.layers, args.steps + args.warmup))
    layers = [PrefillLayer(cfg, (rank * n_res + i) % N_LAYERS_STACK, keep_host=(i == 0)) for i in range(n_res)]
    ctx = make_ctx(cfg, cfg.S, cfg.l_C, 1)
    Kc = torch.zeros(1, cfg.S, cfg.d_c, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(1, cfg.k, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(1, dtype=torch.int32, device="cuda")
    O = torch.empty(1, cfg.S, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda")
    bufs = (Kc, idx, n_sel, O)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(i, ev=None):
        L = layers[i % n_res]
        ctx.set_compressors(L.wq, None, L.wk, None)
        run_prefill_layer(ctx, cfg, L, bufs, ev, phase=i)

    for i in range(args.warmup):
        one_step(i)
    sync_all()
    ctx.read_profile()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.launch_count
    sampled = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for i in range(args.steps):
        one_step(args.warmup + i, sampled)
    e1.record()
    sync_all()
    ms_total = max_over_ranks(e0.elapsed_time(e1), "cuda" if world > 1 else None)
    clocks = sampler.stop() if rank == 0 else None
    launches = ctx.launch_count - launches0
    assert ctx.last_device_status() == 0
    ms_per_step = ms_total / args.steps
    value = world * cfg.S / (N_LAYERS_STACK * ms_per_step * 1e-3)

    # rooflines of the kernels, timed inside the region above on the sampled chunks
    prof = ctx.read_profile()
    by_kernel = kernel_rooflines(prof, sampled, cfg, peaks)
    n_chunks = (cfg.S + cfg.l_C - 1) // cfg.l_C
    att = by_kernel.get("attend_tc_kernel", {"achieved": 0.0, "frac_sustained": 0.0, "frac_burst": 0.0, "launches": 0})
    att_ms = prof.get("attend_tc_kernel", (0, 0.0))[1]
    roofline = {"bound": "tensor", "kernel": "attend_tc_kernel (key-list splits merged inside the kernel)",
                "achieved": att["achieved"], "peak": peaks["tflops_sustained"],
                "unit": "TFLOP/s", "frac": att["frac_sustained"], "frac_sustained": att["frac_sustained"],
                "frac_burst": att["frac_burst"], "peak_burst": peaks["tflops_burst"],
                "traffic": ATTEND_TC_DRAM_BYTES,
                "traffic_unit": "bytes per attend_tc_kernel launch (ncu, profiles/dram_bytes_per_kernel.txt)",
                "peak_source": peaks["source"] + " bf16: sustained (a kernel inside a long step) and burst (the clocks "
                               "sampled during the run decide which applies: at the maximum SM clock, the burst one)",
                "share_of_step": att_ms * (args.steps * n_chunks / max(1, len(sampled))) / ms_total,
                "launches": att["launches"],
                "sampling": "CUDA events around every kernel of 1 chunk in %d, positions moving with the step; an "
                            "event-bracketed launch runs alone, so the kernel's early phase (rows of I and L, normally "
                            "beside the selection kernel) counts in full and share_of_step overstates its part of a "
                            "pipelined step" % PROFILE_EVERY}

    # host time to enqueue a chunk (three library calls + the side-stream bookkeeping), GPU queue empty at the start
    torch.cuda.synchronize()
    probe = cfg.with_(S=64 * cfg.l_C)
    h0 = time.perf_counter()
    run_prefill_layer(ctx, probe, layers[0], bufs)
    host_us_per_chunk = 1e6 * (time.perf_counter() - h0) / 64
    torch.cuda.synchronize()

    # end to end: host inputs and outputs
    L0 = layers[0]
    caches = (torch.zeros_like(L0.K), torch.zeros_like(L0.V))
    g_rows = E2E_GROUP * cfg.l_C
    stage = [(torch.empty(1, g_rows, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda"),
              torch.empty(1, g_rows, cfg.H_G, cfg.d, dtype=torch.bfloat16, device="cuda"),
              torch.empty(1, g_rows, cfg.H_G, cfg.d, dtype=torch.bfloat16, device="cuda"),
              torch.empty(1, g_rows, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda")) for _ in range(2)]
    streams = tuple(torch.cuda.Stream() for _ in range(3))
    O_host = torch.empty(cfg.S, cfg.H, cfg.d, dtype=torch.bfloat16).pin_memory()
    ctx.set_compressors(L0.wq, None, L0.wk, None)
    run_prefill_layer_e2e(ctx, cfg, L0, bufs, caches, stage, O_host, streams)
    sync_all()
    n_e2e = max(1, min(2, args.steps))
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(n_e2e):
        run_prefill_layer_e2e(ctx, cfg, L0, bufs, caches, stage, O_host, streams)
    t1.record()
    sync_all()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1), "cuda" if world > 1 else None) / n_e2e
    h2d = cfg.S * (cfg.d_H + 2 * cfg.d_G) * 2
    d2h = cfg.S * cfg.d_H * 2
    e2e = {"value": world * cfg.S / (N_LAYERS_STACK * e2e_ms * 1e-3), "unit": "tokens/s",
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms}
    del caches, stage, layers, streams
    ctx.close()
    torch.cuda.empty_cache()

    # decode workload (config c3)
    decode = None
    if not args.no_decode:
        cfg3 = syn.get_config("c3")
        us, byts, lps, dprof = time_decode(cfg3, args.decode_steps, rank)
        us = max_over_ranks(us, "cuda" if world > 1 else None)
        gbs = byts / (us * 1e-6) / 1e9
        decode = {"workload": "c3: 8 sequences x 131072 cached tokens, 1 query each, k=4096 l_L=2048 l_I=128",
                  "us_per_step": us, "steps": args.decode_steps, "launches_per_step": lps,
                  "kernels_isolated": dprof,
                  "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": gbs / peaks["hbm_gbs"], "traffic": DECODE_STEP_DRAM_BYTES,
                               "traffic_unit": "bytes per decode step, all kernels (ncu, profiles/dram_bytes_per_kernel.txt)",
                               "algorithmic_bytes_per_step": byts, "peak_source": peaks["source"] + " copy"}}

    # secondary prefill workloads (rank 0's figures are reported; every rank runs them so that the
    # ranks stay in step)
    legs = {}
    if not args.no_legs:
        for name in ("c2", "c4"):
            legs["prefill_" + name] = time_prefill_leg(name, 2, peaks)
        legs["extensions"] = time_extensions(peaks)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    # CPU oracle on a bounded sample of the same workload
    toks, secs, what = oracle_sample(cfg, 0, [13, 255])
    cpu = {"value": toks / secs / N_LAYERS_STACK, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
           "sample": what + "; per-token time extrapolated to the 32-layer stack"}
    line = {
        "metric": "esa_prefill_tokens_per_s_128k", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(cfg), "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "roofline_by_kernel": by_kernel, "host_us_per_chunk": host_us_per_chunk,
        "cpu_baseline": cpu, "decode": decode,
        "per_layer_tokens_per_s": world * cfg.S / (ms_per_step * 1e-3),
    }
    line.update(legs)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="esa", choices=["esa", "reference"])
    ap.add_argument("--layers", type=int, default=3, help="distinct layers' data kept resident")
    ap.add_argument("--decode-steps", type=int, default=256)
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the secondary prefill workloads (c2, c4)")
    ap.add_argument("--profile-case", choices=["prefill", "decode"],
                    help="run a small self-ending case of every kernel of one step (for ncu captures) and exit")
    ap.add_argument("--profile-t", type=int, default=65536, help="tokens cached before the profiled chunk / step")
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    cfg = syn.get_config("c5")
    if args.profile_case:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py --profile-case needs a CUDA device")
        profile_case(args)
        return
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the ESA path has no CPU fallback "
                             "(use --impl reference for the CPU oracle)")
        run_esa(args, cfg)


if __name__ == "__main__":
    main()
