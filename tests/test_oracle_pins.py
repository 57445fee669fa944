"""Pins for the CPU oracle: every function is checked against something other
than itself -- brute-force loops on tiny inputs, library routines it reduces to
in a special case, closed forms the paper prints, and invariants of Eq. 4."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import esa_oracle as orc
import esa_synth as syn

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def rand_bf16(g, *shape, scale=1.0):
    return syn.bf16_bits_to_f64(syn.to_bf16_bits((scale * g.standard_normal(shape)).astype(np.float32)))


# ------------------------------------------------------------------ rounding
def test_bf16_round_matches_library_conversion():
    g = rng(0)
    x32 = (g.standard_normal(20000) * np.exp(g.uniform(-20, 20, 20000))).astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = orc.bf16_round(x32.astype(np.float64))
    assert np.array_equal(got, want)


def test_bf16_round_ties_to_even_and_no_double_rounding():
    assert orc.bf16_round(np.array([1.0 + 2.0 ** -8]))[0] == 1.0                 # midpoint -> even (1.0)
    assert orc.bf16_round(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6  # midpoint -> even
    # just above a midpoint by less than an fp32 ulp: rounding via fp32 first would tie down to 1.0
    assert orc.bf16_round(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1.0 + 2.0 ** -7
    assert orc.bf16_round(np.array([-3.0, 0.0, 0.5]))[1] == 0.0


def test_synth_bf16_bits_roundtrip_is_library_rne():
    g = rng(1)
    x = g.standard_normal(5000).astype(np.float32)
    bits = syn.to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    assert np.array_equal(syn.bf16_bits_to_f32(bits), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


# ----------------------------------------------------------------- partition
@pytest.mark.parametrize("t,l_I,l_L,exp", [
    (0, 4, 8, (0, 0)), (3, 4, 8, (3, 3)), (4, 4, 8, (4, 4)), (10, 4, 8, (4, 4)),
    (12, 4, 8, (4, 4)), (13, 4, 8, (4, 5)), (100, 4, 8, (4, 92)),
])
def test_partition_cases(t, l_I, l_L, exp):
    assert orc.partition(t, l_I, l_L) == exp


def test_partition_invariants():
    for t in range(0, 60):
        for l_I in (0, 1, 5):
            for l_L in (0, 3, 20):
                i_end, m_end = orc.partition(t, l_I, l_L)
                assert 0 <= i_end <= m_end <= t
                assert i_end == min(l_I, t)
                if t >= l_I + l_L:
                    assert t - m_end == l_L and m_end - i_end == t - l_I - l_L
                else:
                    assert m_end == i_end          # no middle tokens yet


# ------------------------------------------------------------------ compress
def test_compress_is_plain_matrix_product_bruteforce():
    g = rng(2)
    X = rand_bf16(g, 5, 12)
    W = rand_bf16(g, 3, 12, scale=0.3)
    b = g.standard_normal(3)
    want = np.empty((5, 3))
    for n in range(5):
        for j in range(3):
            acc = 0.0
            for i in range(12):
                acc += X[n, i] * W[j, i]
            want[n, j] = acc + b[j]
    got = orc.compress(X, W, b)
    # the exact sums agree to fp64 rounding; the oracle then rounds to bf16
    ref = torch.from_numpy(want.astype(np.float32)).to(torch.bfloat16).double().numpy()
    assert np.array_equal(got, ref)


def test_compress_no_bias_equals_zero_bias_and_bias_shifts():
    g = rng(3)
    X, W = rand_bf16(g, 7, 16), rand_bf16(g, 4, 16)
    assert np.array_equal(orc.compress(X, W), orc.compress(X, W, np.zeros(4)))
    big = orc.compress(X, W, np.full(4, 64.0))
    assert np.all(big > orc.compress(X, W))


def test_gqa_folding_identity():
    g = rng(4)
    H, H_G, d, dp, n = 8, 2, 4, 5, 9
    K = g.standard_normal((n, H_G, d))
    Wfull = g.standard_normal((dp, H * d))
    K_rep = np.repeat(K, H // H_G, axis=1).reshape(n, H * d)     # kv head j serves query heads j*g .. j*g+g-1
    lhs = K_rep @ Wfull.T
    rhs = K.reshape(n, H_G * d) @ orc.fold_gqa(Wfull, H, H_G, d).T
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------- scores / aggregation
def brute_scores(qc, kc):
    S = np.zeros((qc.shape[0], kc.shape[0]), np.float32)
    for c in range(qc.shape[0]):
        for m in range(kc.shape[0]):
            acc = 0.0
            for i in range(qc.shape[1]):
                acc += qc[c, i] * kc[m, i]
            S[c, m] = np.float32(acc)
    return S


def brute_aggregate(S):
    l_C, l_M = S.shape
    out = np.empty(l_M, np.float32)
    for m in range(l_M):
        best = None
        for c in range(l_C):
            rmax = max(S[c, mm] for mm in range(l_M))
            v = np.float32(S[c, m]) - np.float32(rmax)
            best = v if best is None or v > best else best
        out[m] = best
    return out


def test_scores_and_aggregate_bruteforce():
    g = rng(5)
    qc, kc = rand_bf16(g, 6, 8), rand_bf16(g, 17, 8)
    S = orc.scores(qc, kc)
    assert S.dtype == np.float32 and S.shape == (6, 17)
    assert np.array_equal(S, brute_scores(qc, kc))
    assert np.array_equal(orc.aggregate(S), brute_aggregate(S))


def test_aggregate_invariants():
    g = rng(6)
    S = g.standard_normal((9, 40)).astype(np.float32)
    s = orc.aggregate(S)
    assert np.all(s <= 0) and s.max() == 0.0
    # every query's arg-max token scores exactly zero
    for c in range(S.shape[0]):
        assert s[np.argmax(S[c])] == 0.0
    assert not np.any(np.signbit(s[s == 0.0]))


def test_decode_shift_invariance_of_selection():
    g = rng(7)
    raw = g.integers(-1000, 1000, size=(1, 300)).astype(np.float32)      # exact in fp32
    k = 37
    sel = orc.topk(orc.aggregate(raw), k)
    brute = sorted(sorted(range(300), key=lambda m: (-raw[0, m], m))[:k])
    assert sel.tolist() == brute


def test_selection_invariant_under_power_of_two_query_scale():
    g = rng(8)
    qc, kc = rand_bf16(g, 5, 16), rand_bf16(g, 200, 16)
    a, _, _ = orc.select(qc, kc, 20, 2)
    b, _, _ = orc.select(qc * 8.0, kc, 20, 2)
    assert np.array_equal(a, b)


# ------------------------------------------------------------------- pooling
@pytest.mark.parametrize("eps", [0, 1, 3, 5])
@pytest.mark.parametrize("n", [1, 2, 7, 64])
def test_pool_equals_library_maxpool(eps, n):
    g = rng(100 + eps + n)
    s = g.standard_normal(n).astype(np.float32)
    want = F.max_pool1d(torch.from_numpy(s)[None, None], kernel_size=2 * eps + 1, stride=1,
                        padding=eps)[0, 0].numpy() if eps > 0 else s
    got = orc.proximity_pool(s, eps)
    assert np.array_equal(got, want)
    assert np.all(got >= s)


def test_pool_window_bruteforce_clipped_to_middle():
    g = rng(9)
    s = g.standard_normal(23).astype(np.float32)
    eps, l_I = 3, 4                                      # absolute token j = l_I + index
    got = orc.proximity_pool(s, eps)
    l_M = s.shape[0]
    for j in range(l_I, l_I + l_M):
        lo, hi = max(j - eps, l_I), min(j + eps, l_I + l_M - 1)
        assert got[j - l_I] == max(s[w - l_I] for w in range(lo, hi + 1))


def test_pool_commutes_with_max_over_queries():
    g = rng(10)
    S = g.standard_normal((7, 50)).astype(np.float32)
    r = S.max(axis=1, keepdims=True)
    a = orc.proximity_pool(orc.aggregate(S), 3)
    b = np.max(np.stack([orc.proximity_pool((S - r)[c], 3) for c in range(7)]), axis=0)
    assert np.array_equal(a, b)


# --------------------------------------------------------------------- top-k
def test_topk_bruteforce_with_ties():
    g = rng(11)
    sp = g.integers(0, 6, size=200).astype(np.float32)          # many exact ties
    for k in (1, 5, 50, 199, 200, 300):
        want = sorted(sorted(range(200), key=lambda m: (-sp[m], m))[:min(k, 200)])
        assert orc.topk(sp, k).tolist() == want


def test_topk_all_equal_takes_first_k():
    assert orc.topk(np.zeros(50, np.float32), 7).tolist() == list(range(7))


def test_topk_prefers_larger_score_then_lower_index():
    sp = np.array([-1, 0, -1, 0, -2, 0], np.float32)
    assert orc.topk(sp, 2).tolist() == [1, 3]
    assert orc.topk(sp, 4).tolist() == [0, 1, 3, 5]
    assert orc.topk(sp, 5).tolist() == [0, 1, 2, 3, 5]


# ----------------------------------------------------------------- attention
def sdpa_ref(Q_C, K, V, visible_abs, scale):
    """Library attention with an explicit boolean mask over absolute positions."""
    l_C, H, d = Q_C.shape
    g = H // K.shape[1]
    q = torch.from_numpy(Q_C).permute(1, 0, 2)[None]                          # [1,H,l_C,d]
    k = torch.from_numpy(K).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    v = torch.from_numpy(V).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    o = F.scaled_dot_product_attention(q, k, v, attn_mask=torch.from_numpy(visible_abs)[None, None], scale=scale)
    return o[0].permute(1, 0, 2).numpy()


def make_qkv(g, t, l_C, H, H_G, d):
    return rand_bf16(g, l_C, H, d), rand_bf16(g, t + l_C, H_G, d), rand_bf16(g, t + l_C, H_G, d)


def test_attend_all_middle_selected_is_textbook_causal_attention():
    g = rng(12)
    t, l_C, H, H_G, d = 45, 6, 4, 2, 8
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    p = orc.EsaParams(l_I=3, l_L=10, k=10 ** 6, eps=1)
    i_end, m_end = orc.partition(t, p.l_I, p.l_L)
    got = orc.attend(Q, K, V, np.arange(i_end, m_end), t, p)
    vis = np.zeros((l_C, t + l_C), bool)
    for c in range(l_C):
        vis[c, : t + c + 1] = True
    want = sdpa_ref(Q, K, V, vis, 1.0 / math.sqrt(d))
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)
    # is_causal flavour of the library call (bottom-right aligned by construction here: pad queries)
    q = torch.from_numpy(np.concatenate([np.zeros((t, H, d)), Q])).permute(1, 0, 2)[None]
    k = torch.from_numpy(K).repeat_interleave(H // H_G, dim=1).permute(1, 0, 2)[None]
    v = torch.from_numpy(V).repeat_interleave(H // H_G, dim=1).permute(1, 0, 2)[None]
    full = F.scaled_dot_product_attention(q, k, v, is_causal=True)[0].permute(1, 0, 2).numpy()[t:]
    assert np.allclose(got, full, rtol=1e-10, atol=1e-12)


def test_attend_subset_matches_library_with_explicit_mask():
    g = rng(13)
    t, l_C, H, H_G, d = 60, 5, 6, 3, 4
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    p = orc.EsaParams(l_I=4, l_L=12, k=7, eps=0, scale=0.37)
    i_end, m_end = orc.partition(t, p.l_I, p.l_L)
    sel = np.sort(g.choice(np.arange(i_end, m_end), size=7, replace=False))
    got = orc.attend(Q, K, V, sel, t, p)
    vis = np.zeros((l_C, t + l_C), bool)
    vis[:, :i_end] = True
    vis[:, sel] = True
    vis[:, m_end:t] = True
    for c in range(l_C):
        vis[c, t: t + c + 1] = True
    assert np.allclose(got, sdpa_ref(Q, K, V, vis, 0.37), rtol=1e-10, atol=1e-12)


# ------------------------------------------- full-dimension and per-head scores
def test_full_dimension_score_is_the_dot_product_of_concatenated_heads():
    """Eq. 3 equals one dot product of the H concatenated heads (keys of a GQA group repeated),
    as Section 3.1 states; also against explicit loops."""
    g = rng(31)
    l_C, l_M, H, H_G, d = 5, 11, 6, 2, 4
    Q = rand_bf16(g, l_C, H, d)
    K = rand_bf16(g, l_M, H_G, d)
    S = orc.scores_full(Q, K)
    K_rep = np.repeat(K, H // H_G, axis=1)                     # [l_M, H, d]
    want = (Q.reshape(l_C, H * d) @ K_rep.reshape(l_M, H * d).T).astype(np.float32)
    assert np.array_equal(S, want)
    brute = np.zeros((l_C, l_M))
    for c in range(l_C):
        for m in range(l_M):
            for h in range(H):
                for i in range(d):
                    brute[c, m] += Q[c, h, i] * K[m, h // (H // H_G), i]
    assert np.allclose(S, brute, rtol=1e-6, atol=1e-6)


def test_per_head_vote_bruteforce_and_reductions():
    g = rng(32)
    l_C, l_M, H, H_G, d = 4, 9, 4, 2, 4
    Q = rand_bf16(g, l_C, H, d)
    K = rand_bf16(g, l_M, H_G, d)
    got = orc.aggregate_per_head(Q, K)
    want = np.full(l_M, -np.inf)
    for h in range(H):
        S_h = np.array([[np.float32(Q[c, h] @ K[m, h // 2]) for m in range(l_M)] for c in range(l_C)], np.float32)
        for m in range(l_M):
            for c in range(l_C):
                want[m] = max(want[m], np.float32(S_h[c, m] - S_h[c].max()))
    assert np.array_equal(got, want.astype(np.float32))
    assert got.max() == 0.0 and np.all(got <= 0)
    # with a single head the vote and the summed score coincide
    Q1, K1 = Q[:, :1], K[:, :1]
    assert np.array_equal(orc.aggregate_per_head(Q1, K1), orc.aggregate(orc.scores_full(Q1, K1)))
    sel_u, sp_u = orc.select_full(Q1, K1, 3, 1)
    sel_i, sp_i = orc.select_full(Q1, K1, 3, 1, per_head=True)
    assert np.array_equal(sel_u, sel_i) and np.array_equal(sp_u, sp_i)


def test_compression_with_an_orthonormal_basis_reproduces_the_full_scores():
    """When the two compressors are the same orthonormal basis of the whole space (d' = d_H), the
    compressed score q' . k' (Eq. 6) is the full-dimension score (Eq. 3), so both selections agree
    and the recall is 1.  Entries are small integers so that every step is exact."""
    g = rng(33)
    l_C, l_M, H, d = 3, 40, 2, 4
    Q = np.round(4 * g.standard_normal((l_C, H, d)))
    K = np.round(4 * g.standard_normal((l_M, H, d)))
    P = np.eye(H * d)[g.permutation(H * d)]                    # a permutation: orthonormal, exact in bf16
    qc, kc = orc.compress(Q.reshape(l_C, -1), P), orc.compress(K.reshape(l_M, -1), P)
    sel_c, sp_c, _ = orc.select(qc, kc, 7, 1)
    sel_f, sp_f = orc.select_full(Q, K, 7, 1)
    assert np.array_equal(sp_c, sp_f) and np.array_equal(sel_c, sel_f)
    assert orc.recall(sel_c, sel_f) == 1.0
    assert orc.recall(np.array([1, 2, 3]), np.array([2, 3, 4, 5])) == 0.5


def test_attention_by_parts_equals_single_softmax():
    """Algorithm 1: a causal part on [L, C] and a non-causal part on [I, M_k], merged by the
    softmax of their log-normalisers, equal one softmax over the union; so does any other cut."""
    g = rng(14)
    t, l_C, H, H_G, d = 80, 7, 4, 1, 8
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    Q *= 4.0                                        # spread the two log-normalisers apart
    p = orc.EsaParams(l_I=5, l_L=16, k=9, eps=1)
    i_end, m_end = orc.partition(t, p.l_I, p.l_L)
    sel = np.sort(g.choice(np.arange(i_end, m_end), size=9, replace=False))
    want = orc.attend(Q, K, V, sel, t, p)
    assert np.allclose(want, orc.attend_by_parts(Q, K, V, sel, t, p), rtol=1e-10, atol=1e-12)
    assert np.allclose(want, orc.attend_by_parts(Q, K, V, sel, t, p, cuts=[3, 20, 33]), rtol=1e-10, atol=1e-12)
    # no far keys at all (chunk 0): the near part alone
    Q0, K0, V0 = make_qkv(g, 0, l_C, H, H_G, d)
    assert np.allclose(orc.attend(Q0, K0, V0, np.zeros(0, np.int64), 0, p),
                       orc.attend_by_parts(Q0, K0, V0, np.zeros(0, np.int64), 0, p), rtol=1e-10, atol=1e-12)


def test_merge_weights_are_the_normalised_exponentials_of_the_log_normalisers():
    """The merge weights written out without the max subtraction (safe here: small values)."""
    g = rng(21)
    o1, o2 = g.standard_normal((5, 3)), g.standard_normal((5, 3))
    l1, l2 = g.standard_normal(5), g.standard_normal(5)
    se = np.exp(np.stack([l1, l2]))
    fac = se / se.sum(axis=0)
    want = o1 * fac[0][:, None] + o2 * fac[1][:, None]
    assert np.allclose(orc.merge_softmax_parts([(o1, l1), (o2, l2)]), want, rtol=1e-12, atol=1e-14)
    # an empty part (log-normaliser -inf) carries no weight
    assert np.allclose(orc.merge_softmax_parts([(o1, l1), (o2, np.full(5, -np.inf))]), o1)


def test_two_position_attention_bruteforce():
    """Section 3.2 / Algorithm 1 with distinct tensors: far-position queries and keys for
    [I, M_k], near-position ones for [L, C], checked against explicit loops (two softmax
    normalisers per row and the merge), and against ``attend`` with the same arguments."""
    g = rng(22)
    t, l_C, H, H_G, d = 40, 5, 4, 2, 8
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    Qg = rand_bf16(g, l_C, H, d)
    Kg = rand_bf16(g, t + l_C, H_G, d)
    p = orc.EsaParams(l_I=3, l_L=9, k=6, eps=0)
    i_end, m_end = orc.partition(t, p.l_I, p.l_L)
    sel = np.sort(g.choice(np.arange(i_end, m_end), size=6, replace=False))
    scale = 1.0 / math.sqrt(d)
    far = list(range(i_end)) + sel.tolist()
    want = np.zeros((l_C, H, d))
    for c in range(l_C):
        near = list(range(m_end, t + c + 1))
        for h in range(H):
            kv = h // (H // H_G)
            lf = [scale * float(Qg[c, h] @ Kg[j, kv]) for j in far]
            ln = [scale * float(Q[c, h] @ K[j, kv]) for j in near]
            zf, zn = sum(math.exp(x) for x in lf), sum(math.exp(x) for x in ln)
            of = sum(math.exp(x) * V[j, kv] for x, j in zip(lf, far)) / zf
            on = sum(math.exp(x) * V[j, kv] for x, j in zip(ln, near)) / zn
            want[c, h] = (zf * of + zn * on) / (zf + zn)
    got = orc.attend(Q, K, V, sel, t, p, Q_global=Qg, K_global=Kg)
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)
    assert np.allclose(orc.attend_by_parts(Q, K, V, sel, t, p, Q_global=Qg, K_global=Kg), want, rtol=1e-10, atol=1e-12)
    # identical tensors for both positions give the one-position result
    assert np.allclose(orc.attend(Q, K, V, sel, t, p, Q_global=Q, K_global=K), orc.attend(Q, K, V, sel, t, p))
    # and a different far query really changes the output
    assert not np.allclose(got, orc.attend(Q, K, V, sel, t, p))


def test_every_initial_local_and_current_key_is_attended():
    g = rng(15)
    t, l_C, H, H_G, d = 50, 4, 2, 1, 4
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    p = orc.EsaParams(l_I=3, l_L=8, k=5, eps=0)
    i_end, m_end = orc.partition(t, p.l_I, p.l_L)
    sel = np.arange(i_end + 2, i_end + 7)
    base = orc.attend(Q, K, V, sel, t, p)
    always = list(range(i_end)) + list(range(m_end, t))
    for j in always + sel.tolist():
        V2 = V.copy()
        V2[j] += 1.0
        diff = np.abs(orc.attend(Q, K, V2, sel, t, p) - base).max(axis=(1, 2))
        assert np.all(diff > 0), f"key {j} must carry weight for every query"
    unselected = [j for j in range(i_end, m_end) if j not in set(sel.tolist())]
    V2 = V.copy()
    V2[unselected] += 1.0
    assert np.array_equal(orc.attend(Q, K, V2, sel, t, p), base)
    # causality inside C: key t+u changes queries c >= u only
    for u in range(l_C):
        V2 = V.copy()
        V2[t + u] += 1.0
        diff = np.abs(orc.attend(Q, K, V2, sel, t, p) - base).max(axis=(1, 2))
        assert np.all(diff[:u] == 0) and np.all(diff[u:] > 0)


def test_gqa_head_mapping():
    g = rng(16)
    t, l_C, H, H_G, d = 20, 3, 4, 2, 4
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    p = orc.EsaParams(l_I=2, l_L=4, k=3, eps=0)
    base = orc.attend(Q, K, V, np.array([5, 6, 9]), t, p)
    V2 = V.copy()
    V2[:, 1] += 1.0                                  # kv head 1 serves query heads 2,3
    out = orc.attend(Q, K, V2, np.array([5, 6, 9]), t, p)
    assert np.array_equal(out[:, :2], base[:, :2]) and np.all(np.abs(out[:, 2:] - base[:, 2:]) > 0.5)


# ------------------------------------------------------------- the whole step
def test_step_composition_and_index_invariants():
    g = rng(17)
    t, l_C, H, H_G, d, dc = 150, 8, 4, 2, 8, 4
    Q, K, V = make_qkv(g, t, l_C, H, H_G, d)
    Wq = orc.bf16_round(g.standard_normal((dc, H * d)) / math.sqrt(H * d))
    Wk = orc.bf16_round(g.standard_normal((dc, H_G * d)) / math.sqrt(H_G * d))
    p = orc.EsaParams(l_I=4, l_L=20, k=16, eps=2)
    res = orc.esa_step(Q, K, V, Wq, Wk, p, t)
    i_end, m_end = orc.partition(t, p.l_I, p.l_L)
    sel = res.sel_abs
    assert len(sel) == 16 and len(set(sel.tolist())) == 16 and np.all(np.diff(sel) > 0)
    assert sel.min() >= i_end and sel.max() < m_end
    # same result from the cached compressed keys and from brute-force pieces
    Kc = orc.compress(K.reshape(t + l_C, -1), Wk)
    res2 = orc.esa_step(Q, K, V, Wq, Wk, p, t, Kc=Kc)
    assert np.array_equal(res2.sel_abs, sel) and np.array_equal(res2.O, res.O)
    S = brute_scores(res.qc, Kc[i_end:m_end])
    sp = orc.proximity_pool(brute_aggregate(S), p.eps)
    want = sorted(sorted(range(m_end - i_end), key=lambda m: (-sp[m], m))[:16])
    assert (sel - i_end).tolist() == want
    # early chunks: no middle tokens -> plain causal attention
    res0 = orc.esa_step(Q, K[: 10 + l_C], V[: 10 + l_C], Wq, Wk, p, 10)
    assert len(res0.sel_abs) == 0
    vis = np.zeros((l_C, 10 + l_C), bool)
    for c in range(l_C):
        vis[c, : 10 + c + 1] = True
    assert np.allclose(res0.O, sdpa_ref(Q, K[: 10 + l_C], V[: 10 + l_C], vis, 1 / math.sqrt(d)), rtol=1e-10, atol=1e-12)


def test_k_not_below_lM_selects_all_middle():
    g = rng(18)
    t, l_C = 40, 2
    Q, K, V = make_qkv(g, t, l_C, 2, 1, 4)
    W = orc.bf16_round(g.standard_normal((2, 8)))
    Wk = orc.bf16_round(g.standard_normal((2, 4)))
    p = orc.EsaParams(l_I=2, l_L=8, k=30, eps=1)
    res = orc.esa_step(Q, K, V, W, Wk, p, t)
    assert res.sel_abs.tolist() == list(range(2, 32))


# --------------------------------------------------------------- accounting
def read_golden():
    vals = {}
    with open(os.path.join(GOLDEN, "paper_closed_forms.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, val = line.split()[:2]
                vals[name] = float(val)
    return vals


def test_paper_closed_forms():
    gold = read_golden()
    d_H, H, dc, d_G = 4096, 32, 128, 1024
    r_limit = (2 * dc + 1) / (4 * d_H + 3 * H)
    assert round(100 * r_limit, 2) == gold["reduction_ratio_percent"]
    assert 100 * orc.cache_overhead(dc, d_G) == gold["cache_overhead_percent"]
    # the oracle's per-step counts approach the printed limit as l_M grows
    l_C, l_I, l_L, k = 512, 128, 4096, 2048
    for l_M, tol in ((10 ** 6, 0.02), (10 ** 8, 2e-4)):
        comp, sel, sparse = orc.flops_esa_step(d_H, H, dc, l_C, l_I, l_M, l_L, k)
        full = orc.flops_full_attention(d_H, H, l_C, l_I + l_M + l_L + l_C)
        assert abs((comp + sel + sparse) / full - r_limit) < tol
    comp, sel, sparse = orc.flops_esa_step(d_H, H, dc, 1, 0, 1000, 0, 0)
    assert comp == 2 * 2 * d_H * dc + 2 * dc and sel == 2 * 1000 * dc + 1000
    assert sparse == (4 * d_H + 3 * H) * 1


# ------------------------------------------------ planted-needle acceptance
def _needle_recall(cfg, layer, span):
    plan = syn.needle_plan(cfg, layer)
    c = int(plan.aligned_chunk[span])
    t = c * cfg.l_C
    wq, wk = syn.compressor_weights(cfg, layer)
    Wq, Wk = orc.bf16_round(wq), orc.bf16_round(wk)
    Q = syn.bf16_bits_to_f64(syn.qkv_rows(cfg, "q", t, t + cfg.l_C, layer))
    K = syn.bf16_bits_to_f64(syn.qkv_rows(cfg, "k", 0, t + cfg.l_C, layer))
    p = orc.EsaParams(cfg.l_I, cfg.l_L, cfg.k, cfg.eps)
    res = orc.esa_step(Q, K, None, Wq, Wk, p, t, do_attend=False)
    chosen = set(res.sel_abs.tolist())
    hit = tot = 0
    for i in plan.spans_in_chunk(c):
        for tok in plan.needle_tokens(i):
            if res.i_end <= tok < res.m_end:
                tot += 1
                hit += tok in chosen
    return hit, tot, len(chosen)


def test_needles_are_selected_small_context():
    cfg = syn.get_config("c5").with_(S=32768, l_C=256, l_L=1024, k=1024)
    for span in (0, 13, 31):
        hit, tot, n = _needle_recall(cfg, 0, span)
        assert tot >= 16 and hit == tot and n == cfg.k


def test_needles_are_selected_full_size_chunk():
    cfg = syn.get_config("c5")
    hit, tot, n = _needle_recall(cfg, 1, 7)
    assert tot >= 16 and hit == tot and n == cfg.k


# ------------------------------------------------------- compressor fitting (Eq. 7)
def _fit_problem(g, n=6, H=4, H_G=2, d=3, dc=2):
    from oracle import esa_fit_oracle as fo
    Q = g.standard_normal((n, H, d))
    K = g.standard_normal((n, H_G, d))
    P = {"Wq": 0.3 * g.standard_normal((dc, H * d)), "bq": 0.1 * g.standard_normal(dc),
         "Wk": 0.3 * g.standard_normal((dc, H_G * d)), "bk": 0.1 * g.standard_normal(dc)}
    return fo, Q, K, P


def test_fit_target_is_the_full_dimension_score():
    g = rng(41)
    fo, Q, K, _ = _fit_problem(g)
    T = fo.fold_heads(Q, K.shape[1]) @ K.reshape(K.shape[0], -1).T
    assert np.allclose(T, orc.scores_full(Q, K).astype(np.float64), rtol=1e-6, atol=1e-6)


def test_fit_gradients_match_finite_differences():
    g = rng(42)
    fo, Q, K, P = _fit_problem(g)
    loss, dWq, dbq, dWk, dbk = fo.loss_and_grads(Q, K, P["Wq"], P["bq"], P["Wk"], P["bk"])
    grads = {"Wq": dWq, "bq": dbq, "Wk": dWk, "bk": dbk}
    h = 1e-6
    for name in grads:
        flat = P[name].reshape(-1)
        for i in range(0, flat.size, max(1, flat.size // 5)):
            old = flat[i]
            flat[i] = old + h
            lp = fo.loss_and_grads(Q, K, P["Wq"], P["bq"], P["Wk"], P["bk"])[0]
            flat[i] = old - h
            lm = fo.loss_and_grads(Q, K, P["Wq"], P["bq"], P["Wk"], P["bk"])[0]
            flat[i] = old
            assert abs((lp - lm) / (2 * h) - grads[name].reshape(-1)[i]) <= 1e-5 * max(1.0, abs(grads[name].reshape(-1)[i])), name


def test_first_adam_step_moves_by_lr_against_the_gradient_sign():
    g = rng(43)
    fo, Q, K, P = _fit_problem(g)
    before = {k: v.copy() for k, v in P.items()}
    grads = dict(zip(("Wq", "bq", "Wk", "bk"), fo.loss_and_grads(Q, K, P["Wq"], P["bq"], P["Wk"], P["bk"])[1:]))
    st = fo.AdamState(lr=5e-4)
    fo.fit_step(P, Q, K, st)
    for name in P:
        assert np.allclose(P[name] - before[name], -5e-4 * np.sign(grads[name]), rtol=1e-4, atol=1e-9)


def test_fit_reaches_near_zero_loss_when_the_data_lie_in_a_small_subspace():
    """Queries and keys confined to a d'-dimensional subspace (one head, no grouping) admit exact
    compressors -- the projection on that subspace -- so the loss can be driven towards zero."""
    from oracle import esa_fit_oracle as fo
    g = rng(44)
    D, dc, n = 12, 3, 16
    basis = np.linalg.qr(g.standard_normal((D, dc)))[0]             # [D, dc] orthonormal columns
    P = {"Wq": 0.5 * g.standard_normal((dc, D)), "bq": np.zeros(dc), "Wk": 0.5 * g.standard_normal((dc, D)), "bk": np.zeros(dc)}
    st = fo.AdamState(lr=2e-2)
    first = last = None
    for it in range(1500):
        Q = (g.standard_normal((n, dc)) @ basis.T)[:, None, :]
        K = (g.standard_normal((n, dc)) @ basis.T)[:, None, :]
        loss = fo.fit_step(P, Q, K, st)
        first = loss if first is None else first
        last = loss
    assert last < 1e-3 * first
