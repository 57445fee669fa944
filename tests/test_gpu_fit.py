"""Compressor fitting (Eq. 7) on the GPU against the float64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import esa_synth as syn
from oracle import esa_fit_oracle as fo
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


def _run(cfg, n, steps, lr, seed):
    import paper_2502_14477_b200 as esa
    ec = esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps, 1, 1, 16)
    fit = esa.EsaFit(ec, n, lr)
    wq, wk = syn.compressor_weights(cfg)
    bq, bk = syn.compressor_bias(cfg)
    bq, bk = 0.01 * bq, 0.01 * bk
    fit.set_weights(wq, bq, wk, bk)
    P = {"Wq": wq.astype(np.float64), "bq": bq.astype(np.float64), "Wk": wk.astype(np.float64), "bk": bk.astype(np.float64)}
    st = fo.AdamState(lr=lr)
    loss_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    losses = []
    for it in range(steps):
        # a batch of (q, k) pairs: seeded rows of the workload's queries and keys
        r0 = (seed + it) * n
        Qb, Kb = syn.qkv_rows(cfg, "q", r0, r0 + n), syn.qkv_rows(cfg, "k", r0, r0 + n)
        fit.step(hp.bits_to_torch(Qb).contiguous(), hp.bits_to_torch(Kb).contiguous(), loss_dev)
        want = fo.fit_step(P, syn.bf16_bits_to_f64(Qb), syn.bf16_bits_to_f64(Kb), st)
        losses.append((float(loss_dev[0]), want))
    got = dict(zip(("Wq", "bq", "Wk", "bk"), fit.get_weights()))
    fit.close()
    return losses, got, P


@pytest.mark.parametrize("name,n,steps", [("c1", 128, 40), ("c1", 37, 10), ("c2", 128, 6)])
def test_fit_steps_follow_the_oracle(name, n, steps):
    cfg = syn.get_config(name)
    lr = 5e-4
    losses, got, want = _run(cfg, n, steps, lr, seed=3)
    for it, (a, b) in enumerate(losses):
        assert abs(a - b) <= 2e-4 * abs(b), f"loss of step {it}: {a} against {b}"
    for key in want:
        d = np.abs(got[key].astype(np.float64) - want[key])
        tol = 2e-6 + 1e-4 * np.abs(want[key])
        # fp32 against float64: a gradient that is zero to rounding can flip the sign of an early Adam step
        assert (d > tol).mean() <= 2e-3, f"{key}: {(d > tol).mean():.2e} of the elements differ"
        assert d.max() <= 2.5 * lr, f"{key}: largest difference {d.max():.3e}"


def test_fitting_lowers_the_loss_and_raises_the_recall_of_the_selection():
    """A short fit on the mixture workload: the loss falls, and the selection made with the fitted
    compressors recovers more of the full-dimension selection (Fig. 3's recall) than the one made
    with the random initial compressors."""
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config("c5").with_(S=16384)
    n, steps = 128, 300
    ec = esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps, cfg.l_C, 1, cfg.S)
    fit = esa.EsaFit(ec, n, 5e-4)
    wq, wk = syn.compressor_weights(cfg)
    fit.set_weights(wq, None, wk, None)
    Qall = hp.bits_to_torch(syn.qkv_rows(cfg, "q", 0, 8192))
    Kall = hp.bits_to_torch(syn.qkv_rows(cfg, "k", 0, 8192))
    loss_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(0)
    losses = []
    for it in range(steps):
        iq = torch.randint(0, 8192, (n,), device="cuda", generator=g)
        ik = torch.randint(0, 8192, (n,), device="cuda", generator=g)
        fit.step(Qall[iq].contiguous(), Kall[ik].contiguous(), loss_dev)
        losses.append(float(loss_dev[0]))
    assert np.mean(losses[-10:]) < 0.7 * np.mean(losses[:10])
    Wq2, bq2, Wk2, bk2 = fit.get_weights()
    fit.close()
    # recall of the compressed selection at one chunk, before and after the fit
    t, l_C = cfg.S - cfg.l_C, cfg.l_C
    seq = hp.DeviceSeq(cfg, max_tokens=cfg.S, B=1)
    seq.fill_kv(0, cfg.S)
    Q = hp.bits_to_torch(syn.qkv_rows(cfg, "q", t, t + l_C))[None].contiguous()
    rec = []
    for weights in ((wq, None, wk, None), (Wq2, bq2, Wk2, bk2)):
        ctx = esa.Esa(ec)
        ctx.set_compressors(*weights)
        for r0 in range(0, t, 4096):
            ctx.compress_keys(seq.K[:, r0: min(t, r0 + 4096)].contiguous(), seq.Kc, [r0])
        ctx.select(Q, seq.Kc, [t], seq.idx, seq.n_sel, sync=True)
        sel_c = seq.idx[0, : int(seq.n_sel[0])].clone()
        ctx.select_full(Q, seq.K, [t], seq.idx, seq.n_sel, sync=True)
        sel_f = seq.idx[0, : int(seq.n_sel[0])]
        rec.append(float(torch.isin(sel_f, sel_c).float().mean()))
        ctx.close()
    print(f"loss {np.mean(losses[:10]):.1f} -> {np.mean(losses[-10:]):.1f}; recall {rec[0]:.3f} -> {rec[1]:.3f}")
    assert rec[1] > rec[0]
