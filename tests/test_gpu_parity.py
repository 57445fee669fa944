"""GPU-vs-oracle parity of the ESA step, through the C ABI (ctypes binding).

Small cases compare every output element; the full-size workloads compare
sampled chunks / decode steps (each step is a pure function of its inputs, so a
chunk can be checked without running the ones before it)."""
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


def fill_kc_gpu(ctx, seq: hp.DeviceSeq, upto: int, step: int = 4096):
    """k' for rows [0, upto) of every sequence, by the library itself."""
    for r0 in range(0, upto, step):
        r1 = min(upto, r0 + step)
        ctx.compress_keys(seq.K[:, r0:r1].contiguous(), seq.Kc, [r0] * seq.B)


def oracle_kc_bits(cfg, K64: np.ndarray, Wk) -> np.ndarray:
    kc = orc.compress(K64.reshape(K64.shape[0], -1), Wk)
    return syn.to_bf16_bits(kc.astype(np.float32))


def run_step_gpu(ctx, seq: hp.DeviceSeq, Q: torch.Tensor, t_list, do_compress=True):
    B, l_C = Q.shape[0], Q.shape[1]
    if do_compress:
        Knew = torch.stack([seq.K[b, t_list[b]: t_list[b] + l_C] for b in range(B)]).contiguous()
        ctx.compress_keys(Knew, seq.Kc, t_list)
    ctx.select(Q, seq.Kc, t_list, seq.idx, seq.n_sel)
    O = torch.empty_like(Q)
    ctx.attend(Q, seq.K, seq.V, t_list, seq.idx, seq.n_sel, O)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 0
    n = seq.n_sel.cpu().numpy()
    idx = seq.idx.cpu().numpy()
    return [idx[b, : n[b]].astype(np.int64) for b in range(B)], O


def attend_on_oracle_selection(ctx, seq, Q, t_list, b, res):
    """Re-runs esa_attend with sequence b's selection replaced by the oracle's (the other sequences
    keep whatever the buffers hold) and returns O[b]: used when the kernel's index set differs from
    the oracle's by in-band tokens, so that the attention output is still compared like for like."""
    n = len(res.sel_abs)
    seq.idx[b, :n] = torch.from_numpy(res.sel_abs.astype(np.int32)).cuda()
    seq.n_sel[b] = n
    O = torch.empty_like(Q)
    ctx.attend(Q, seq.K, seq.V, t_list, seq.idx, seq.n_sel, O, sync=True)
    assert ctx.last_device_status() == 0
    return O[b]


# --------------------------------------------------------------- compression
@pytest.mark.parametrize("name,n_new,with_bias", [("c1", 128, False), ("c1", 37, True), ("c1", 13, True), ("c1", 7, True), ("c1", 1, False), ("c2", 512, False),
                                                   ("c2", 1, False), ("c2", 8, True), ("c2", 700, True)])
def test_compress_keys_parity(name, n_new, with_bias):
    cfg = syn.get_config(name).with_(S=2048, n_decode=0)
    bias = syn.compressor_bias(cfg) if with_bias else None
    ctx = hp.make_esa(cfg, max_tokens=2048, max_chunk=1024, max_batch=2, bias=bias)
    _, _, Wq, Wk = hp.oracle_weights(cfg)
    B = 2
    n_prev = [5, 1000]
    Kbits = [syn.qkv_rows(cfg, "k", 0, n_new, 0, b) for b in range(B)]
    Knew = torch.stack([hp.bits_to_torch(x) for x in Kbits])
    kc = torch.zeros(B, 2048, cfg.d_c, dtype=torch.bfloat16, device="cuda")
    ctx.compress_keys(Knew, kc, n_prev, sync=True)
    for b in range(B):
        X = syn.bf16_bits_to_f64(Kbits[b]).reshape(n_new, -1)
        hp.check_compressed(kc[b, n_prev[b]: n_prev[b] + n_new], X, Wk, None if bias is None else bias[1],
                            what=f"{name} b{b}")
        # rows outside the appended range stay untouched
        assert float(kc[b, : n_prev[b]].abs().sum()) == 0.0
        assert float(kc[b, n_prev[b] + n_new:].abs().sum()) == 0.0


def test_query_sized_compression_through_compress_keys():
    """Eq. 5 at the query compressor's shape (d_in = H d = 4096, 512 rows) through the public key
    entry point: with H_G = H the key compressor has the query compressor's shape, and the
    weights installed for it are the query compressor's."""
    cfg = syn.get_config("c2").with_(H_G=32, S=1024, n_decode=0)
    import paper_2502_14477_b200 as esa
    ctx = esa.Esa(esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, cfg.l_I, cfg.l_L, cfg.k, cfg.eps, 512, 1, 1024))
    wq, _ = syn.compressor_weights(cfg)
    bias = syn.compressor_bias(cfg)
    ctx.set_compressors(wq, bias[0], wq, bias[1])
    Wq = orc.bf16_round(wq)
    Xb = syn.qkv_rows(syn.get_config("c2"), "q", 0, 512)                  # [512, 32, 128]
    kc = torch.zeros(1, 1024, cfg.d_c, dtype=torch.bfloat16, device="cuda")
    ctx.compress_keys(hp.bits_to_torch(Xb)[None].contiguous(), kc, [100], sync=True)
    hp.check_compressed(kc[0, 100:612], syn.bf16_bits_to_f64(Xb).reshape(512, -1), Wq, bias[1], what="query-sized")


def test_append_kv_copies_rows():
    cfg = syn.get_config("c1").with_(S=512, n_decode=0)
    ctx = hp.make_esa(cfg, max_tokens=512, max_batch=3)
    B, n_new = 3, 19
    Knew = torch.randn(B, n_new, cfg.H_G, cfg.d, device="cuda").bfloat16()
    Vnew = torch.randn(B, n_new, cfg.H_G, cfg.d, device="cuda").bfloat16()
    Kc = torch.zeros(B, 512, cfg.H_G, cfg.d, dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    n_prev = [0, 100, 493]
    ctx.append_kv(Knew, Vnew, Kc, Vc, n_prev, sync=True)
    for b in range(B):
        assert torch.equal(Kc[b, n_prev[b]: n_prev[b] + n_new], Knew[b])
        assert torch.equal(Vc[b, n_prev[b]: n_prev[b] + n_new], Vnew[b])
        assert float(Kc[b].abs().sum()) == float(Knew[b].abs().sum())


# ---------------------------------------------- stage-isolated select / attend
def _stage_isolated(cfg, t, l_C, layer=0, eps=None, heads=None, check_scores=True):
    """GPU select fed the ORACLE's compressed keys; GPU attend fed the ORACLE's selection."""
    eps = cfg.eps if eps is None else eps
    p = orc.EsaParams(cfg.l_I, cfg.l_L, cfg.k, eps)
    _, _, Wq, Wk = hp.oracle_weights(cfg, layer)
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1, layer=layer, eps=eps)
    seq = hp.DeviceSeq(cfg, max_tokens=n, layer=layer, B=1)
    seq.fill_kv(0, n)
    K64 = hp.torch_to_f64(seq.K[0])
    V64 = hp.torch_to_f64(seq.V[0])
    Qb = syn.qkv_rows(cfg, "q", t, t + l_C, layer, 0)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    Q64 = syn.bf16_bits_to_f64(Qb)
    Kc64 = orc.compress(K64.reshape(n, -1), Wk)
    seq.Kc[0] = hp.bits_to_torch(syn.to_bf16_bits(Kc64.astype(np.float32)))
    res = orc.esa_step(Q64, K64, V64, Wq, Wk, p, t, Kc=Kc64, heads=heads)
    # select
    ctx.select(Q, seq.Kc, [t], seq.idx, seq.n_sel, sync=True)
    n_sel = int(seq.n_sel[0])
    sel_gpu = seq.idx[0, :n_sel].cpu().numpy().astype(np.int64)
    ndiff = hp.check_index_sets(sel_gpu, res, cfg.k, what=f"{cfg.name} t={t} l_C={l_C} eps={eps}")
    l_M = res.m_end - res.i_end
    if l_M > cfg.k:
        # q' (Eq. 5 for the queries) as the kernel computed it, against the exact product
        qc_gpu = syn.bf16_bits_to_f64(ctx.read_compressed_queries(l_C))
        hp.check_compressed(torch.from_numpy(qc_gpu), Q64.reshape(l_C, -1), Wq, what=f"{cfg.name} t={t} q'")
        if check_scores:
            # s' against the oracle evaluated on the kernel's own q' and the shared k': only the fp32
            # accumulation order differs
            sp_gpu = ctx.read_pooled_scores(0, l_M)
            hp.check_pooled_scores(sp_gpu, qc_gpu, Kc64[res.i_end: res.m_end], cfg.k, eps, what=f"{cfg.name} t={t}")
    # attend on the oracle's selection
    seq.idx[0, : len(res.sel_abs)] = torch.from_numpy(res.sel_abs.astype(np.int32)).cuda()
    seq.n_sel[0] = len(res.sel_abs)
    O = torch.empty_like(Q)
    ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O, sync=True)
    hp.check_attention(O[0], res.O, what=f"{cfg.name} t={t}", heads=heads)
    assert ctx.last_device_status() == 0
    return ndiff


@pytest.mark.parametrize("t,l_C", [(0, 128), (128, 128), (640, 128), (768, 128), (772, 128), (773, 128),
                                   (1536, 128), (3968, 128), (4000, 77), (4096, 1), (4111, 1), (2000, 5)])
def test_c1_stage_isolated(t, l_C):
    _stage_isolated(syn.get_config("c1"), t, l_C)


@pytest.mark.parametrize("eps", [0, 1, 5])
def test_c1_eps_variants(eps):
    _stage_isolated(syn.get_config("c1"), 3968, 128, eps=eps)
    _stage_isolated(syn.get_config("c1"), 4100, 1, eps=eps)


def test_c2_shape_stage_isolated_mid_chunk():
    _stage_isolated(syn.get_config("c2"), 16 * 512, 512, heads=[0, 5, 31])


def test_gqa_group_of_seven_stage_isolated():
    cfg = syn.get_config("c4").with_(S=16384, l_C=256, l_L=1024, k=1024)
    _stage_isolated(cfg, 40 * 256, 256, heads=[0, 6, 7, 27])
    _stage_isolated(cfg, 10000, 1, heads=None)


def test_odd_row_count_through_the_split_merge():
    # l_C * G odd and not a multiple of the row tile: the last row tile is ragged, the parts of the
    # split key list are padded to an even row count, and the merging CTA skips the rows past the end
    cfg = syn.get_config("c4").with_(S=8192, l_C=255, l_L=1024, k=1024)
    _stage_isolated(cfg, 20 * 255, 255, heads=[0, 6, 13, 27], check_scores=False)


def test_all_equal_scores_take_lowest_indices():
    """Identical compressed keys give identical scores: the first k middle tokens win."""
    cfg = syn.get_config("c1")
    t, l_C = 2048, 128
    ctx = hp.make_esa(cfg, max_tokens=t + l_C, max_batch=1)
    kc = torch.ones(1, t + l_C, cfg.d_c, dtype=torch.bfloat16, device="cuda")
    Q = hp.bits_to_torch(syn.qkv_rows(cfg, "q", t, t + l_C))[None].contiguous()
    idx = torch.zeros(1, cfg.k, dtype=torch.int32, device="cuda")
    n_sel = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.select(Q, kc, [t], idx, n_sel, sync=True)
    assert int(n_sel[0]) == cfg.k
    assert idx[0].cpu().tolist() == list(range(cfg.l_I, cfg.l_I + cfg.k))


# ------------------------------------------------------ end to end, config 1
def test_c1_end_to_end_prefill_and_decode():
    cfg = syn.get_config("c1")
    p = hp.oracle_params(cfg)
    _, _, Wq, Wk = hp.oracle_weights(cfg)
    ctx = hp.make_esa(cfg)
    seq = hp.DeviceSeq(cfg)
    n = cfg.max_tokens
    Kb, Vb = syn.qkv_rows(cfg, "k", 0, n), syn.qkv_rows(cfg, "v", 0, n)
    K64, V64 = syn.bf16_bits_to_f64(Kb), syn.bf16_bits_to_f64(Vb)
    Kdev, Vdev = hp.bits_to_torch(Kb), hp.bits_to_torch(Vb)
    Qb = syn.qkv_rows(cfg, "q", 0, n)
    steps = [(t, cfg.l_C) for t in range(0, cfg.S, cfg.l_C)] + [(cfg.S + i, 1) for i in range(cfg.n_decode)]
    total_diff = 0
    for t, l_C in steps:
        Knew, Vnew = Kdev[None, t: t + l_C].contiguous(), Vdev[None, t: t + l_C].contiguous()
        ctx.append_kv(Knew, Vnew, seq.K, seq.V, [t])
        Q = hp.bits_to_torch(Qb[t: t + l_C])[None].contiguous()
        sel, O = run_step_gpu(ctx, seq, Q, [t])
        res = orc.esa_step(syn.bf16_bits_to_f64(Qb[t: t + l_C]), K64[: t + l_C], V64[: t + l_C], Wq, Wk, p, t)
        rep = hp.check_index_sets(sel[0], res, cfg.k, what=f"c1 e2e t={t}")
        total_diff += rep.n_diff
        Ob = attend_on_oracle_selection(ctx, seq, Q, [t], 0, res) if rep else O[0]
        hp.check_attention(Ob, res.O, what=f"c1 t={t}")
    # the library's own compressed-key cache against the exact product
    hp.check_compressed(seq.Kc[0, :n], K64.reshape(n, -1), Wk, what="c1 cache")
    assert total_diff <= 0.01 * cfg.k * len(steps)


# --------------------------------------------- full-size workloads, sampled
def _sampled_prefill(cfg, chunks, layer=0, heads=None):
    p = hp.oracle_params(cfg)
    _, _, Wq, Wk = hp.oracle_weights(cfg, layer)
    t_max = max(chunks) * cfg.l_C
    n = t_max + cfg.l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_batch=1, layer=layer)
    seq = hp.DeviceSeq(cfg, max_tokens=n, layer=layer, B=1)
    seq.fill_kv(0, n)
    fill_kc_gpu(ctx, seq, n)
    K64 = hp.torch_to_f64(seq.K[0])
    V64 = hp.torch_to_f64(seq.V[0])
    out = []
    for c in chunks:
        t = c * cfg.l_C
        Qb = syn.qkv_rows(cfg, "q", t, t + cfg.l_C, layer, 0)
        Q = hp.bits_to_torch(Qb)[None].contiguous()
        sel, O = run_step_gpu(ctx, seq, Q, [t], do_compress=False)
        res = orc.esa_step(syn.bf16_bits_to_f64(Qb), K64[: t + cfg.l_C], V64[: t + cfg.l_C], Wq, Wk, p, t, heads=heads)
        rep = hp.check_index_sets(sel[0], res, cfg.k, what=f"{cfg.name} layer {layer} chunk {c}")
        # attention is compared on the oracle's own selection unless the sets agree exactly
        Ob = attend_on_oracle_selection(ctx, seq, Q, [t], 0, res) if rep else O[0]
        hp.check_attention(Ob, res.O, what=f"{cfg.name} chunk {c}", heads=heads)
        out.append((sel[0], res))
    return out


def test_c2_sampled_chunks():
    # first chunk, last chunk without middle tokens, first with l_M > k, a middle one, the last
    _sampled_prefill(syn.get_config("c2"), [0, 4, 13, 40, 63], heads=[0, 9, 18, 31])


def test_c4_sampled_chunks():
    cfg = syn.get_config("c4")
    _sampled_prefill(cfg, [5, 13, 255], heads=[0, 13, 27])


@pytest.mark.parametrize("layer", [0, 3, 17, 31])
def test_c5_needle_chunks(layer):
    cfg = syn.get_config("c5")
    plan = syn.needle_plan(cfg, layer)
    span = int(np.argmax(plan.aligned_chunk))          # the latest aligned chunk of this layer
    chunk = int(plan.aligned_chunk[span])
    last = cfg.S // cfg.l_C - 1
    chunks = [chunk] if chunk == last else [chunk, last]
    out = _sampled_prefill(cfg, chunks, layer=layer, heads=[0, 17])
    sel, res = out[0]
    chosen = set(sel.tolist())
    for i in plan.spans_in_chunk(chunk):
        for tok in plan.needle_tokens(i):
            if res.i_end <= tok < res.m_end:
                assert tok in chosen, f"needle token {tok} of span {i} not selected"


def test_c3_decode_steps():
    cfg = syn.get_config("c3")
    p = hp.oracle_params(cfg)
    _, _, Wq, Wk = hp.oracle_weights(cfg)
    ctx = hp.make_esa(cfg)
    seq = hp.DeviceSeq(cfg)
    n = cfg.max_tokens
    seq.fill_kv(0, n)
    fill_kc_gpu(ctx, seq, cfg.S)
    steps = (0, 1, 127, 255)
    runs = {}
    for step in steps:
        t = cfg.S + step
        # k' of the tokens decoded before this step (rows S..t) are appended by the library
        if step > 0:
            upto = [cfg.S] * cfg.B
            ctx.compress_keys(seq.K[:, cfg.S: t].contiguous(), seq.Kc, upto)
        Q = seq.q_rows(t, t + 1).contiguous()
        sel, O = run_step_gpu(ctx, seq, Q, [t] * cfg.B)
        runs[step] = (Q, sel, O.clone())
    # every sequence at every sampled step (bf16 values are exact in float32: the oracle converts
    # the rows it gathers to float64 itself)
    for b in range(cfg.B):
        K32 = seq.K[b].float().cpu().numpy()
        V32 = seq.V[b].float().cpu().numpy()
        Kc_or = orc.compress(K32.reshape(n, -1), Wk)
        hp.check_compressed(seq.Kc[b, : cfg.S + steps[-1]], K32[: cfg.S + steps[-1]].reshape(cfg.S + steps[-1], -1).astype(np.float64),
                            Wk, what=f"c3 seq {b} cache")
        for step in steps:
            t = cfg.S + step
            Q, sel, O = runs[step]
            res = orc.esa_step(hp.torch_to_f64(Q[b]), K32[: t + 1], V32[: t + 1], Wq, Wk, p, t, Kc=Kc_or)
            rep = hp.check_index_sets(sel[b], res, cfg.k, what=f"c3 step {step} seq {b}")
            Ob = attend_on_oracle_selection(ctx, seq, Q, [t] * cfg.B, b, res) if rep else O[b]
            hp.check_attention(Ob, res.O, what=f"c3 step {step} seq {b}")


# ------------------------------------------- batch of ragged sequences, d' = 64
def test_batch_of_ragged_sequences_dc64():
    """Two sequences at different positions in one call (different partitions, one with every middle
    token selected and one scored), compressed dimension 64: the tensor-core kernels' other
    instantiation and the per-sequence bookkeeping."""
    cfg = syn.get_config("c2").with_(H=8, H_G=2, d_c=64, l_C=256, l_I=16, l_L=512, k=512, S=6144, B=2)
    p = hp.oracle_params(cfg)
    _, _, Wq, Wk = hp.oracle_weights(cfg)
    l_C = cfg.l_C
    t_list = [768, 5000]                       # |M| = 240 (all selected) and 4472 (scored)
    n = max(t_list) + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=2)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=2)
    seq.fill_kv(0, n)
    fill_kc_gpu(ctx, seq, n, step=1024)
    Q = torch.stack([hp.bits_to_torch(syn.qkv_rows(cfg, "q", t, t + l_C, 0, b)) for b, t in enumerate(t_list)]).contiguous()
    sel, O = run_step_gpu(ctx, seq, Q, t_list, do_compress=False)
    for b, t in enumerate(t_list):
        K64 = hp.torch_to_f64(seq.K[b, : t + l_C])
        V64 = hp.torch_to_f64(seq.V[b, : t + l_C])
        res = orc.esa_step(hp.torch_to_f64(Q[b]), K64, V64, Wq, Wk, p, t)
        rep = hp.check_index_sets(sel[b], res, cfg.k, what=f"ragged seq {b}")
        Ob = attend_on_oracle_selection(ctx, seq, Q, t_list, b, res) if rep else O[b]
        hp.check_attention(Ob, res.O, what=f"ragged seq {b}")
        hp.check_compressed(seq.Kc[b, : t], K64[:t].reshape(t, -1), Wk, what=f"ragged seq {b} cache")


def test_compress_keys_on_a_side_stream_matches_the_serial_order():
    """esa_compress_keys uses none of the context's workspace: run beside select/attend on another
    stream (ordered only against the selection that first reads its rows) it must give the very
    bits of the one-stream order."""
    cfg = syn.get_config("c1")
    n = 2048
    outs = []
    for use_side in (False, True):
        ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=cfg.l_C, max_batch=1)
        seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
        seq.fill_kv(0, n)
        O = torch.zeros(1, n, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda")
        idx_log = []
        main = torch.cuda.current_stream()
        side = torch.cuda.Stream()
        side.wait_stream(main)
        prev = None
        for t in range(0, n, cfg.l_C):
            Q = seq.q_rows(t, t + cfg.l_C)
            Knew = seq.K[:, t: t + cfg.l_C].contiguous()
            if use_side:
                side.wait_stream(main)          # Knew was produced on the main stream
                with torch.cuda.stream(side):
                    ctx.compress_keys(Knew, seq.Kc, [t])
                    done = torch.cuda.Event()
                    done.record(side)
                Knew.record_stream(side)
                if prev is not None:
                    main.wait_event(prev)
                prev = done
            else:
                ctx.compress_keys(Knew, seq.Kc, [t])
            ctx.select(Q, seq.Kc, [t], seq.idx, seq.n_sel)
            ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O[:, t: t + cfg.l_C])
            idx_log.append((seq.idx.clone(), seq.n_sel.clone()))
        main.wait_stream(side)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == 0
        outs.append((seq.Kc.clone(), O, idx_log))
    (kc0, o0, l0), (kc1, o1, l1) = outs
    assert torch.equal(kc0, kc1)
    assert torch.equal(o0, o1)
    for (i0, n0), (i1, n1) in zip(l0, l1):
        assert torch.equal(n0, n1)
        k = int(n0[0])
        assert torch.equal(i0[0, :k], i1[0, :k])


# ------------------------------- full-dimension and per-head selection (Eq. 3, Section 4.3)
class _FullResult:
    """What check_index_sets reads, for a selection made on full-dimension scores."""

    def __init__(self, sel_abs, pooled, rowmax, i_end, m_end):
        self.sel_abs, self.pooled, self.rowmax, self.i_end, self.m_end = sel_abs, pooled, rowmax, i_end, m_end


def _select_full_case(cfg, t, l_C, per_head, layer=0):
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1, layer=layer)
    seq = hp.DeviceSeq(cfg, max_tokens=n, layer=layer, B=1)
    seq.fill_kv(0, n)
    Qb = syn.qkv_rows(cfg, "q", t, n, layer)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    Q64 = syn.bf16_bits_to_f64(Qb)
    i_end, m_end = orc.partition(t, cfg.l_I, cfg.l_L)
    K_M = hp.torch_to_f64(seq.K[0, i_end:m_end])
    sel, sp = orc.select_full(Q64, K_M, cfg.k, cfg.eps, per_head=per_head)
    ctx.select_full(Q, seq.K, [t], seq.idx, seq.n_sel, per_head=per_head, sync=True)
    assert ctx.last_device_status() == 0
    n_sel = int(seq.n_sel[0])
    sel_gpu = seq.idx[0, :n_sel].cpu().numpy().astype(np.int64)
    S_abs_max = float(np.abs(orc.scores_full(Q64, K_M)).max()) if m_end > i_end else 0.0
    res = _FullResult(sel + i_end, sp, np.array([S_abs_max], np.float32), i_end, m_end)
    hp.check_index_sets(sel_gpu, res, cfg.k, what=f"{cfg.name} full{'/per-head' if per_head else ''} t={t} l_C={l_C}")
    if m_end - i_end > cfg.k:
        # pooled scores within the fp32 accumulation bound of the d_H-long sums (the bound of the summed score
        # also covers each head's own shorter sum)
        K_rep = np.repeat(K_M, cfg.H // cfg.H_G, axis=1).reshape(m_end - i_end, -1)
        tol, _ = hp.score_error_bound(Q64.reshape(l_C, -1), K_rep, cfg.eps)
        got = ctx.read_pooled_scores(0, m_end - i_end).astype(np.float64)
        err = np.abs(got - sp.astype(np.float64))
        assert np.all(err <= tol), f"pooled full-dimension scores off by {err.max():.3e} (bound {tol[np.argmax(err)]:.3e})"
        assert got.max() == 0.0 and np.all(got <= 0)
    return sel_gpu


@pytest.mark.parametrize("per_head", [False, True])
@pytest.mark.parametrize("t,l_C", [(3968, 128), (4000, 77), (4100, 1), (2000, 5), (640, 128)])
def test_select_full_c1(t, l_C, per_head):
    _select_full_case(syn.get_config("c1"), t, l_C, per_head)


@pytest.mark.parametrize("per_head", [False, True])
def test_select_full_llama_shape(per_head):
    _select_full_case(syn.get_config("c2"), 8192, 512, per_head)
    _select_full_case(syn.get_config("c2"), 9000, 1, per_head)


def test_recall_of_the_compressed_selection_against_the_full_dimension_one():
    """Fig. 3's metric on the mixture-with-needles workload: the share of the full-dimension
    selection (Eq. 3) that the compressed selection (Eq. 6) also picks.  The kernels' recall equals
    the oracle's (random-init compressors: the number itself is not a quality claim)."""
    cfg = syn.get_config("c5")
    p = hp.oracle_params(cfg)
    _, _, Wq, Wk = hp.oracle_weights(cfg)
    t, l_C = 32 * 512, 512
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_batch=1)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    fill_kc_gpu(ctx, seq, t)
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    ctx.select(Q, seq.Kc, [t], seq.idx, seq.n_sel, sync=True)
    sel_c = seq.idx[0, : int(seq.n_sel[0])].cpu().numpy().astype(np.int64)
    ctx.select_full(Q, seq.K, [t], seq.idx, seq.n_sel, sync=True)
    sel_f = seq.idx[0, : int(seq.n_sel[0])].cpu().numpy().astype(np.int64)
    Q64, K64 = syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0])
    i_end, m_end = orc.partition(t, cfg.l_I, cfg.l_L)
    res = orc.esa_step(Q64, K64, K64, Wq, Wk, p, t, do_attend=False)
    sel_f_or, _ = orc.select_full(Q64, K64[i_end:m_end], cfg.k, cfg.eps)
    want = orc.recall(res.sel_abs, sel_f_or + i_end)
    got = orc.recall(sel_c, sel_f)
    print(f"recall of the compressed selection: kernels {got:.4f}, oracle {want:.4f}")
    assert abs(got - want) <= 2.0 / cfg.k


# ------------------------------------------------ two-position attention (Section 3.2)
def _two_position_case(cfg, t, l_C, heads=None, use_qfar=True, use_kfar=True, n_sel=None, seed=0):
    """esa_attend_two_position against the oracle: I and M_k attended with a second encoding of the
    queries and keys (stand-ins: independent seeded tensors), L and C with the first."""
    p = hp.oracle_params(cfg)
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Qfb = syn.qkv_rows(cfg, "q", t, n, layer=7)              # the far-position encoding of the same tokens
    Kfb = syn.qkv_rows(cfg, "k", 0, n, layer=7)
    Q, Qf = hp.bits_to_torch(Qb)[None].contiguous(), hp.bits_to_torch(Qfb)[None].contiguous()
    Kf = hp.bits_to_torch(Kfb)[None].contiguous()
    i_end, m_end = orc.partition(t, cfg.l_I, cfg.l_L)
    l_M = m_end - i_end
    kk = min(cfg.k, l_M) if n_sel is None else n_sel
    g = np.random.default_rng(seed)
    sel = np.sort(g.choice(np.arange(i_end, m_end), size=kk, replace=False)) if kk else np.zeros(0, np.int64)
    seq.idx[0, :kk] = torch.from_numpy(sel.astype(np.int32)).cuda()
    seq.n_sel[0] = kk
    O = torch.full_like(Q, float("nan"))
    ctx.attend_two_position(Q, Qf if use_qfar else None, seq.K, Kf if use_kfar else None, seq.V, [t], seq.idx, seq.n_sel, O,
                            sync=True)
    assert ctx.last_device_status() == 0
    want = orc.attend(syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0]), hp.torch_to_f64(seq.V[0]), sel, t, p, heads=heads,
                      Q_global=syn.bf16_bits_to_f64(Qfb) if use_qfar else None,
                      K_global=syn.bf16_bits_to_f64(Kfb) if use_kfar else None)
    hp.check_attention(O[0], want, what=f"two-position {cfg.name} t={t} l_C={l_C}", heads=heads)
    # the far tensors matter: where I and M_k are a fair share of the list, the one-position result differs
    if (use_qfar or use_kfar) and 4 * (i_end + kk) >= n - m_end:
        one = orc.attend(syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0]), hp.torch_to_f64(seq.V[0]), sel, t, p, heads=heads)
        hs = heads if heads is not None else slice(None)
        assert np.abs(one[:, hs] - want[:, hs]).max() > 2 * hp.ATT_MAX_ABS


@pytest.mark.parametrize("t,l_C", [(3968, 128), (3000, 77), (4100, 1), (2000, 5), (640, 128), (0, 128), (300, 1)])
def test_two_position_attention_c1(t, l_C):
    _two_position_case(syn.get_config("c1"), t, l_C)


def test_two_position_attention_partial_tensors_and_ragged_far_part():
    cfg = syn.get_config("c1")
    _two_position_case(cfg, 3968, 128, use_kfar=False)                 # far queries only
    _two_position_case(cfg, 3968, 128, use_qfar=False)                 # far keys only
    _two_position_case(cfg, 3968, 128, n_sel=201)                      # |I| + |M_k| = 205: the far part ends inside a tile
    _two_position_case(cfg, 4100, 1, n_sel=201)
    _two_position_case(cfg, 4000, 9, n_sel=37)


def test_two_position_attention_llama_shape_and_group_of_seven():
    _two_position_case(syn.get_config("c2"), 16 * 512, 512, heads=[0, 5, 31])
    _two_position_case(syn.get_config("c2"), 9000, 1)
    cfg = syn.get_config("c4").with_(S=16384, l_C=256, l_L=1024, k=1024)
    _two_position_case(cfg, 40 * 256, 256, heads=[0, 6, 7, 27])
    _two_position_case(cfg, 10000, 1)


# ------------------------------------------------ host-resident K/V (appendix "Model Loading")
@pytest.mark.parametrize("name,t,l_C,n_sel", [("c1", 3968, 128, None), ("c1", 4100, 1, None), ("c1", 2000, 5, 100),
                                               ("c1", 300, 128, None), ("c2", 8192, 512, None), ("c2", 9000, 1, None)])
def test_attention_with_host_resident_kv(name, t, l_C, n_sel):
    """The K/V cache lives in pinned host memory; the attended rows are staged on the device by the
    library's gather kernel.  Same bits as esa_attend on device-resident copies, and within the attention tolerance
    of the oracle."""
    cfg = syn.get_config(name)
    p = hp.oracle_params(cfg)
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    K_host = seq.K.cpu().pin_memory()
    V_host = seq.V.cpu().pin_memory()
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    i_end, m_end = orc.partition(t, cfg.l_I, cfg.l_L)
    kk = min(cfg.k, m_end - i_end) if n_sel is None else n_sel
    g = np.random.default_rng(5)
    sel = np.sort(g.choice(np.arange(i_end, m_end), size=kk, replace=False)) if kk else np.zeros(0, np.int64)
    seq.idx[0, :kk] = torch.from_numpy(sel.astype(np.int32)).cuda()
    seq.n_sel[0] = kk
    stage_rows = cfg.l_I + cfg.k + cfg.l_L + l_C
    K_stage = torch.zeros(1, stage_rows, cfg.H_G, cfg.d, dtype=torch.bfloat16, device="cuda")
    V_stage = torch.zeros_like(K_stage)
    O_host = torch.full_like(Q, float("nan"))
    ctx.attend_host_kv(Q, K_host, V_host, [t], seq.idx, seq.n_sel, K_stage, V_stage, O_host, sync=True)
    O_dev = torch.empty_like(Q)
    ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O_dev, sync=True)
    assert ctx.last_device_status() == 0
    # (neither call follows a selection of its step, so neither attends the older rows early: the same sums in the
    # same order)
    assert torch.equal(O_host, O_dev)
    want = orc.attend(syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0]), hp.torch_to_f64(seq.V[0]), sel, t, p,
                      heads=[0, cfg.H - 1])
    hp.check_attention(O_host[0], want, what=f"host K/V {name} t={t} l_C={l_C}", heads=[0, cfg.H - 1])
    # a stage that cannot hold the list is refused before anything is launched
    import paper_2502_14477_b200 as esa
    small = torch.zeros(1, 16, cfg.H_G, cfg.d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(esa.EsaError) as e:
        ctx.attend_host_kv(Q, K_host, V_host, [t], seq.idx, seq.n_sel, small, small.clone(), O_host, sync=True)
    assert e.value.status == 3


# ------------------------------------------------------- device-side safety nets
@pytest.mark.parametrize("name,t,l_C", [("c1", 3968, 128), ("c1", 4100, 1), ("c1", 300, 128), ("c1", 2000, 5), ("c1", 700, 77),
                                        ("c2", 8192, 512), ("c2", 9000, 1)])
def test_attention_that_follows_its_selection_attends_the_older_rows_early(name, t, l_C):
    """esa_attend enqueued right after the esa_select of its step attends the rows of I and L (older than the chunk, so
    independent of the selection) ahead of its wait for the selection kernel; a call that follows no selection takes
    the list in order after the wait.  The same set of keys either way: both results are within the attention
    tolerance of the oracle on the kernel's own selection.  They differ from each other by the rounding of P and of the
    result: P is rounded to bf16 against the running maximum of the moment, which depends on the order, and a
    relative error of 2^-9 on every weight moves a weighted mean of V by up to 2^-9 max|V| on each side, however small
    the mean itself is; the result is then rounded to bf16 once more."""
    cfg = syn.get_config(name)
    p = hp.oracle_params(cfg)
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    fill_kc_gpu(ctx, seq, n)
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    O_early = torch.full_like(Q, float("nan"))
    torch.cuda.synchronize()
    ctx.select(Q, seq.Kc, [t], seq.idx, seq.n_sel)
    ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O_early)       # armed by the selection just enqueued
    torch.cuda.synchronize()
    O_plain = torch.full_like(Q, float("nan"))
    ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O_plain, sync=True)
    assert ctx.last_device_status() == 0
    # a selection enqueued on another stream arms nothing: the attention call takes the list in order after its wait
    other = torch.cuda.Stream()
    idx2, n_sel2 = torch.zeros_like(seq.idx), torch.zeros_like(seq.n_sel)
    other.wait_stream(torch.cuda.current_stream())
    ctx.select(Q, seq.Kc, [t], idx2, n_sel2, stream=other)
    other.synchronize()
    assert torch.equal(idx2, seq.idx) and torch.equal(n_sel2, seq.n_sel)
    O_other = torch.full_like(Q, float("nan"))
    ctx.attend(Q, seq.K, seq.V, [t], idx2, n_sel2, O_other, sync=True)
    assert torch.equal(O_other, O_plain)
    a, b = O_early.float(), O_plain.float()
    v_max = float(seq.V[0, :n].float().abs().max())
    bound = 2.0 ** -8 * v_max + 2.0 ** -8 * torch.maximum(a.abs(), b.abs())
    assert bool(((a - b).abs() <= bound).all()), (float((a - b).abs().max()), v_max)
    assert float((a - b).abs().mean()) <= hp.ATT_MEAN_ABS
    sel = seq.idx[0, : int(seq.n_sel[0])].cpu().numpy().astype(np.int64)
    want = orc.attend(syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0]), hp.torch_to_f64(seq.V[0]), sel, t, p,
                      heads=[0, cfg.H - 1])
    hp.check_attention(O_early[0], want, what=f"early {name} t={t} l_C={l_C}", heads=[0, cfg.H - 1])
    hp.check_attention(O_plain[0], want, what=f"plain {name} t={t} l_C={l_C}", heads=[0, cfg.H - 1])


@pytest.mark.parametrize("t,l_C", [(3000, 1), (3000, 5), (2944, 128)])
def test_selected_position_outside_M_is_clamped_and_reported(t, l_C):
    """A stale index buffer must not become a read outside the caches: the position is replaced
    by the nearest one of M, the status word reports ESA_ERR_INDEX, and the next call is clean.
    Covers the decode kernel, the small-chunk kernel and the tensor-core kernel."""
    cfg = syn.get_config("c1")
    p = hp.oracle_params(cfg)
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    i_end, m_end = orc.partition(t, cfg.l_I, cfg.l_L)
    good = np.arange(i_end + 7, i_end + 7 + cfg.k, dtype=np.int64)
    res_O = orc.attend(syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0]), hp.torch_to_f64(seq.V[0]), good, t, p)
    seq.n_sel[0] = cfg.k
    for bad_value in (2 ** 30, -5, m_end, i_end - 1):
        bad = good.copy()
        bad[11] = bad_value
        seq.idx[0] = torch.from_numpy(bad.astype(np.int32)).cuda()
        O = torch.full_like(Q, float("nan"))
        ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O, sync=True)
        assert torch.isfinite(O.float()).all()
        assert ctx.last_device_status() == 8, bad_value
        assert ctx.last_device_status() == 0                      # reading the status clears it
    seq.idx[0] = torch.from_numpy(good.astype(np.int32)).cuda()
    O = torch.empty_like(Q)
    ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O, sync=True)
    assert ctx.last_device_status() == 0
    hp.check_attention(O[0], res_O, what="after a clamped index")


@pytest.mark.parametrize("name,t,l_C,gain", [("c2", 8192, 512, 12.0), ("c2", 8192, 512, 40.0), ("c1", 3968, 128, 12.0),
                                              ("c2", 9000, 1, 12.0)])
def test_attention_with_logits_that_grow_along_the_key_list(name, t, l_C, gain):
    """Keys scaled up along the positions, so that the largest logit of a row lies tens to hundreds of
    powers of two above the one its running maximum was set on.  The prefill kernel takes its exponentials
    against the standing maximum and looks for a tile's own maximum only when the tile's sum overflows its
    limit: this drives that path (and the rescaling of the accumulator behind it); the other kernels run the
    same rows through their ordinary online softmax.  Compared with the oracle like every other attention."""
    cfg = syn.get_config(name)
    p = hp.oracle_params(cfg)
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1)
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    # K rows grow linearly with the position, to `gain` times their size at the end of the cache (bf16 again)
    ramp = (1.0 + (gain - 1.0) * torch.arange(n, device="cuda", dtype=torch.float32) / n).view(1, n, 1, 1)
    seq.K.copy_((seq.K.float() * ramp).to(torch.bfloat16))
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    i_end, m_end = orc.partition(t, cfg.l_I, cfg.l_L)
    kk = min(cfg.k, m_end - i_end)
    sel = np.sort(np.random.default_rng(11).choice(np.arange(i_end, m_end), size=kk, replace=False))
    seq.idx[0, :kk] = torch.from_numpy(sel.astype(np.int32)).cuda()
    seq.n_sel[0] = kk
    O = torch.full_like(Q, float("nan"))
    ctx.attend(Q, seq.K, seq.V, [t], seq.idx, seq.n_sel, O, sync=True)
    assert ctx.last_device_status() == 0
    heads = [0, cfg.H - 1]
    K64 = hp.torch_to_f64(seq.K[0])
    want = orc.attend(syn.bf16_bits_to_f64(Qb), K64, hp.torch_to_f64(seq.V[0]), sel, t, p, heads=heads)
    # the steep case is only worth its name if the logits of a row really span more than the kernel's limit of 2^64
    q_last = syn.bf16_bits_to_f64(Qb).reshape(l_C, cfg.H, cfg.d)[-1, 0]
    lg = (K64.reshape(n, cfg.H_G, cfg.d)[:, 0] @ q_last) / np.sqrt(cfg.d) * 1.4426950408889634
    if gain >= 40.0:
        assert lg.max() - lg[: cfg.l_I].max() > 64.0, float(lg.max() - lg[: cfg.l_I].max())
    # With logits this steep a row's weight sits on one or two keys, and the bf16 rounding of that weight (up to
    # 2^-9 relative, against a sum kept in fp32) goes straight into the output, times the value: the largest
    # error is bounded relative to the largest value (0.5 %), the mean error by the usual tolerance.
    got = hp.torch_to_f64(O[0])[:, heads]
    err = np.abs(got - want[:, heads])
    vmax = float(np.abs(hp.torch_to_f64(seq.V[0])).max())
    print(f"growing logits {name} t={t} l_C={l_C} x{gain}: max-abs {err.max():.3e} mean-abs {err.mean():.3e} max|V| {vmax:.2f}")
    assert np.isfinite(got).all()
    assert err.max() <= 5e-3 * vmax and err.mean() <= hp.ATT_MEAN_ABS, (float(err.max()), float(err.mean()), vmax)


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """The give-up path of the device-side waits: a wait on a barrier that nothing completes runs
    out after its cycle limit, the kernel returns, the status word says ESA_ERR_TIMEOUT, reading
    it clears it, and the next attention on the same context is correct."""
    cfg = syn.get_config("c1")
    p = hp.oracle_params(cfg)
    t, l_C = 2944, 128
    n = t + l_C
    ctx = hp.make_esa(cfg, max_tokens=n, max_chunk=l_C, max_batch=1)
    ctx.debug_wait_timeout(200_000)                # about 0.1 ms of SM clocks
    torch.cuda.synchronize()
    assert ctx.last_device_status() == 5
    assert ctx.last_device_status() == 0
    seq = hp.DeviceSeq(cfg, max_tokens=n, B=1)
    seq.fill_kv(0, n)
    fill_kc_gpu(ctx, seq, t)
    Qb = syn.qkv_rows(cfg, "q", t, n)
    Q = hp.bits_to_torch(Qb)[None].contiguous()
    sel, O = run_step_gpu(ctx, seq, Q, [t])
    _, _, Wq, Wk = hp.oracle_weights(cfg)
    res = orc.esa_step(syn.bf16_bits_to_f64(Qb), hp.torch_to_f64(seq.K[0]), hp.torch_to_f64(seq.V[0]), Wq, Wk, p, t)
    rep = hp.check_index_sets(sel[0], res, cfg.k, what="after a timed-out wait")
    Ob = attend_on_oracle_selection(ctx, seq, Q, [t], 0, res) if rep else O[0]
    hp.check_attention(Ob, res.O, what="after a timed-out wait")


# ----------------------------------------------------------------- error paths
def test_argument_errors_leave_outputs_untouched():
    import paper_2502_14477_b200 as esa
    cfg = syn.get_config("c1")
    ctx = hp.make_esa(cfg, max_tokens=1024, max_batch=1)
    Q = torch.zeros(1, 128, cfg.H, cfg.d, dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros(1, 1024, cfg.d_c, dtype=torch.bfloat16, device="cuda")
    idx = torch.full((1, cfg.k), -7, dtype=torch.int32, device="cuda")
    n_sel = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(esa.EsaError) as e:
        ctx.select(Q, kc, [1000], idx, n_sel, sync=True)          # 1000 + 128 > max_tokens
    assert e.value.status == 3
    with pytest.raises(esa.EsaError) as e:
        ctx.select(Q, kc, [-1], idx, n_sel, sync=True)
    assert e.value.status == 1
    assert int(idx.min()) == -7 and int(n_sel[0]) == -7
    ctx2 = esa.Esa(esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, 4, 512, 256, 3, 128, 1, 1024))
    with pytest.raises(esa.EsaError) as e:
        ctx2.select(Q, kc, [0], idx, n_sel, sync=True)            # compressors not set
    assert e.value.status == 7
    with pytest.raises(esa.EsaError):
        esa.Esa(esa.EsaConfig(7, 2, 64, 32, 4, 512, 256, 3, 128, 1, 1024))   # H not a multiple of H_G
    # the pooling window of Eq. 8 is taken inside one warp: 2 * eps + 1 <= 31
    with pytest.raises(esa.EsaError) as e:
        esa.Esa(esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, 4, 512, 256, 16, 128, 1, 1024))
    assert e.value.status == 2
    esa.Esa(esa.EsaConfig(cfg.H, cfg.H_G, cfg.d, cfg.d_c, 4, 512, 256, 15, 128, 1, 1024))
