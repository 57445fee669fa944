"""Small, self-ending cases of the library's kernels for ``ncu`` captures.

    python -m paper_2502_14477_b200.profile_cases --case prefill --t 65536 --reps 3
    python -m paper_2502_14477_b200.profile_cases --case decode --cached 131072 --batch 8 --reps 3

Each case holds well under a few GB on the device, uses inputs larger than L2
where DRAM figures matter, and launches every kernel of one ESA step ``reps``
times.  Inputs are N(0,1) bf16 drawn on the device; correctness is the parity
tests' business, not this file's.
"""
from __future__ import annotations

import argparse

import torch

from . import Esa, EsaConfig


def run_prefill(args):
    H, HG, d, dc = args.heads, args.kv_heads, 128, 128
    l_C, t = args.chunk, args.t
    n = t + l_C
    ctx = Esa(EsaConfig(H, HG, d, dc, 128, args.local, args.topk, 3, l_C, 1, n))
    g = torch.Generator(device="cuda").manual_seed(0)
    K = torch.randn(1, n, HG, d, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(1, n, HG, d, device="cuda", dtype=torch.bfloat16, generator=g)
    Q = torch.randn(1, l_C, H, d, device="cuda", dtype=torch.bfloat16, generator=g)
    wq = (torch.randn(dc, H * d, generator=torch.Generator().manual_seed(1)) / (H * d) ** 0.5).numpy()
    wk = (torch.randn(dc, HG * d, generator=torch.Generator().manual_seed(2)) / (HG * d) ** 0.5).numpy()
    ctx.set_compressors(wq, None, wk, None)
    Kc = torch.zeros(1, n, dc, dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, t, 4096):
        r1 = min(t, r0 + 4096)
        ctx.compress_keys(K[:, r0:r1].contiguous(), Kc, [r0])
    idx = torch.zeros(1, args.topk, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(1, dtype=torch.int32, device="cuda")
    O = torch.empty_like(Q)
    torch.cuda.synchronize()
    for _ in range(args.reps):
        ctx.compress_keys(K[:, t:n].contiguous(), Kc, [t])
        ctx.select(Q, Kc, [t], idx, n_sel)
        ctx.attend(Q, K, V, [t], idx, n_sel, O)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    print("prefill case done:", ctx.launch_count, "launches")


def run_decode(args):
    H, HG, d, dc = args.heads, args.kv_heads, 128, 128
    B, S = args.batch, args.cached
    n = S + args.reps + 1
    ctx = Esa(EsaConfig(H, HG, d, dc, 128, args.local, args.topk, 3, 1, B, n))
    g = torch.Generator(device="cuda").manual_seed(0)
    K = torch.randn(B, n, HG, d, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(B, n, HG, d, device="cuda", dtype=torch.bfloat16, generator=g)
    Kc = torch.randn(B, n, dc, device="cuda", dtype=torch.bfloat16, generator=g)
    Q = torch.randn(B, 1, H, d, device="cuda", dtype=torch.bfloat16, generator=g)
    wq = (torch.randn(dc, H * d, generator=torch.Generator().manual_seed(1)) / (H * d) ** 0.5).numpy()
    wk = (torch.randn(dc, HG * d, generator=torch.Generator().manual_seed(2)) / (HG * d) ** 0.5).numpy()
    ctx.set_compressors(wq, None, wk, None)
    idx = torch.zeros(B, args.topk, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(B, dtype=torch.int32, device="cuda")
    O = torch.empty_like(Q)
    torch.cuda.synchronize()
    for i in range(args.reps):
        t = [S + i] * B
        ctx.compress_keys(K[:, S + i: S + i + 1].contiguous(), Kc, t)
        ctx.select(Q, Kc, t, idx, n_sel)
        ctx.attend(Q, K, V, t, idx, n_sel, O)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    print("decode case done:", ctx.launch_count, "launches")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", choices=["prefill", "decode"], required=True)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--chunk", type=int, default=512)
    ap.add_argument("--t", type=int, default=65536, help="tokens cached before the profiled chunk")
    ap.add_argument("--cached", type=int, default=131072)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--local", type=int, default=2048)
    ap.add_argument("--topk", type=int, default=4096)
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    if args.case == "prefill":
        run_prefill(args)
    else:
        run_decode(args)


if __name__ == "__main__":
    main()
