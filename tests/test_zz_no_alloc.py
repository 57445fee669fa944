"""esa_attend_noalloc against esa_attend_async.

The no-allocation entry point exists for callers that cannot allocate device memory while
they run (a serving loop that cannot afford cudaMalloc's device-wide synchronisation, or a
host that has given all device memory to its own pool).  It keeps the split partials in a
fixed array inside the library instead of a context's workspace, so the check is simply that
it reproduces the ordinary entry point -- twice in a row, because the array is shared between
calls and keeps the previous call's contents.  This file sorts last on purpose: a run that
stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

import esa_synth as syn
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


def _case(cfg, B, cached, seed):
    import paper_2502_14477_b200 as esa
    n = cached + 1
    ec = esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps, 1, B, n)
    g = torch.Generator(device="cuda").manual_seed(seed)
    K = torch.randn(B, n, cfg.H_G, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(B, n, cfg.H_G, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
    Q = torch.randn(B, 1, cfg.H, cfg.d, device="cuda", dtype=torch.bfloat16, generator=g)
    # any valid selection will do: k distinct middle positions per sequence
    l_M = cached - cfg.l_L - cfg.l_I
    assert l_M > cfg.k
    idx = torch.stack([torch.sort(torch.randperm(l_M, device="cuda", generator=g)[: cfg.k])[0] + cfg.l_I
                       for _ in range(B)]).to(torch.int32).contiguous()
    n_sel = torch.full((B,), cfg.k, dtype=torch.int32, device="cuda")
    return ec, Q, K, V, idx, n_sel


@pytest.mark.parametrize("name,B,cached", [("c3", 4, 16384), ("c1", 2, 3000)])
def test_noalloc_matches_context_entry_point_twice(name, B, cached):
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config(name)
    for call in range(2):                      # two calls in a row share the fixed scratch array
        ec, Q, K, V, idx, n_sel = _case(cfg, B, cached, seed=10 * call + B)
        ctx = esa.Esa(ec)
        O_ref = torch.empty_like(Q)
        ctx.attend(Q, K, V, [cached] * B, idx, n_sel, O_ref)
        O_new = torch.full_like(Q, float("nan"))
        esa.attend_noalloc(ec, Q, K, V, [cached] * B, idx, n_sel, O_new)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == 0
        got, want = hp.torch_to_f64(O_new), hp.torch_to_f64(O_ref)
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        assert err.max() <= hp.ATT_MAX_ABS and err.mean() <= hp.ATT_MEAN_ABS, (call, err.max(), err.mean())
        ctx.close()


def test_noalloc_rejects_what_does_not_fit():
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config("c3")
    ec, Q, K, V, idx, n_sel = _case(cfg, 1, 8192, seed=3)
    # a prefill-sized chunk has more than 64 rows per key/value head
    Qbig = torch.zeros(1, 128, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(esa.EsaError) as e:
        esa.attend_noalloc(ec, Qbig, K, V, [8192 - 127], idx, n_sel, torch.empty_like(Qbig))
    assert e.value.status == 3
    # the position plus the chunk must fit the cache
    with pytest.raises(esa.EsaError) as e:
        esa.attend_noalloc(ec, Q, K, V, [8193], idx, n_sel, torch.empty_like(Q))
    assert e.value.status == 3
