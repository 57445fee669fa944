"""esa_attend_noalloc against esa_attend_async and against the CPU oracle.

The no-allocation entry point exists for callers that cannot allocate device memory while
they run (a serving loop that cannot afford cudaMalloc's device-wide synchronisation, or a
host that has given all device memory to its own pool).  It keeps the split partials in a
fixed array inside the library instead of a context's workspace, so the check is that it
reproduces the ordinary entry point and the oracle's attention -- twice in a row, because the
array is shared between calls and keeps the previous call's contents.  One case has a single
query per sequence (4 rows per key/value head), one has 8 queries (32 rows: the wider
instantiation, several rows per part of the shared array), and one is a ragged batch of two
sequences of different lengths (the shorter one leaves parts of the key-list split empty).  This file sorts last on purpose: a run that
stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

import esa_synth as syn
from oracle import esa_oracle as orc
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


def _case(cfg, B, cached, seed, l_C=1, t_list=None):
    import paper_2502_14477_b200 as esa
    n = cached + l_C
    t_list = t_list or [cached] * B
    ec = esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps, l_C, B, n)
    g = torch.Generator(device="cuda").manual_seed(seed)
    K = torch.randn(B, n, cfg.H_G, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(B, n, cfg.H_G, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
    Q = torch.randn(B, l_C, cfg.H, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
    # any valid selection will do: distinct middle positions of each sequence, min(k, |M|) of them
    idx = torch.zeros(B, cfg.k, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(B, dtype=torch.int32, device="cuda")
    for b, t in enumerate(t_list):
        l_M = max(0, t - cfg.l_L - cfg.l_I)
        kk = min(cfg.k, l_M)
        if kk:
            idx[b, :kk] = (torch.sort(torch.randperm(l_M, device="cuda", generator=g)[:kk])[0] + cfg.l_I).to(torch.int32)
        n_sel[b] = kk
    return ec, Q, K, V, idx, n_sel, t_list


@pytest.mark.parametrize("name,B,cached,l_C,t_list", [("c3", 4, 16384, 1, None), ("c1", 2, 3000, 1, None),
                                                       ("c3", 2, 12000, 8, None), ("c3", 2, 9000, 8, [9000, 2500])])
def test_noalloc_matches_context_entry_point_and_oracle_twice(name, B, cached, l_C, t_list):
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config(name)
    p = hp.oracle_params(cfg)
    for call in range(2):                      # two calls in a row share the fixed scratch array
        ec, Q, K, V, idx, n_sel, ts = _case(cfg, B, cached, seed=10 * call + B, l_C=l_C, t_list=t_list)
        ctx = esa.Esa(ec)
        O_ref = torch.empty_like(Q)
        ctx.attend(Q, K, V, ts, idx, n_sel, O_ref)
        O_new = torch.full_like(Q, float("nan"))
        esa.attend_noalloc(ec, Q, K, V, ts, idx, n_sel, O_new)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == 0
        got, want = hp.torch_to_f64(O_new), hp.torch_to_f64(O_ref)
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        assert err.max() <= hp.ATT_MAX_ABS and err.mean() <= hp.ATT_MEAN_ABS, (call, err.max(), err.mean())
        # both entry points against the oracle's attention (Eq. 1) on the same selection
        for b, t in enumerate(ts):
            sel = idx[b, : int(n_sel[b])].cpu().numpy().astype(np.int64)
            want_b = orc.attend(hp.torch_to_f64(Q[b]), K[b, : t + l_C].float().cpu().numpy(),
                                V[b, : t + l_C].float().cpu().numpy(), sel, t, p)
            hp.check_attention(O_new[b], want_b, what=f"noalloc {name} call {call} seq {b}")
            hp.check_attention(O_ref[b], want_b, what=f"context {name} call {call} seq {b}")
        ctx.close()


def test_noalloc_rejects_what_does_not_fit():
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config("c3")
    ec, Q, K, V, idx, n_sel, _ = _case(cfg, 1, 8192, seed=3)
    # a prefill-sized chunk has more than 64 rows per key/value head
    Qbig = torch.zeros(1, 128, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(esa.EsaError) as e:
        esa.attend_noalloc(ec, Qbig, K, V, [8192 - 127], idx, n_sel, torch.empty_like(Qbig))
    assert e.value.status == 3
    # the position plus the chunk must fit the cache
    with pytest.raises(esa.EsaError) as e:
        esa.attend_noalloc(ec, Q, K, V, [8193], idx, n_sel, torch.empty_like(Q))
    assert e.value.status == 3
