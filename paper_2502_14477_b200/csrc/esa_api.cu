// C ABI of the ESA library: argument checks, token partition (Section 3.1), workspace
// and launch sequencing.  All arithmetic of the step runs in the kernels.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "esa_internal.h"

using namespace esa;

namespace {

bool config_ok(const esa_config* c) {
    if (!c) return false;
    if (c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->n_q_heads % c->n_kv_heads) return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->d_c != 32 && c->d_c != 64 && c->d_c != 128) return false;
    if (c->l_init < 0 || c->l_local < 0 || c->top_k <= 0 || c->eps < 0 || c->eps > 15) return false;
    if (c->max_chunk <= 0 || c->max_batch <= 0 || c->max_batch > kMaxBatch) return false;
    if (c->max_tokens <= 0 || c->max_tokens >= (int64_t(1) << 31)) return false;
    if ((int64_t)c->n_q_heads * c->head_dim % 64 || (int64_t)c->n_kv_heads * c->head_dim % 64) return false;
    if (!(c->softmax_scale >= 0.f)) return false;
    return true;
}

size_t align_up(size_t x) { return (x + 255) & ~size_t(255); }

struct Layout {
    size_t wq, wk, bq, bk, qc, rkey, rkey_heads, skey, pkey, ghist0, ghist1, cidx, slice_cnt, ticket, att, att_count, status, total;
    size_t att_elems, att_count_elems, slice_stride;
};

Layout make_layout(const esa_config* c) {
    Layout L;
    const size_t dH = (size_t)c->n_q_heads * c->head_dim, dG = (size_t)c->n_kv_heads * c->head_dim;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
    L.wq = take(2 * c->d_c * dH);
    L.wk = take(2 * c->d_c * dG);
    L.bq = take(4 * c->d_c);
    L.bk = take(4 * c->d_c);
    L.qc = take(2 * (size_t)c->max_batch * c->max_chunk * c->d_c);
    L.rkey = take(4 * (size_t)c->max_batch * c->max_chunk);
    L.rkey_heads = take(4 * (size_t)c->max_batch * c->max_chunk * c->n_q_heads);
    L.skey = take(4 * (size_t)c->max_batch * c->max_tokens);
    L.pkey = take(4 * (size_t)c->max_batch * c->max_tokens);
    L.ghist0 = take(4 * (size_t)c->max_batch * 2048);
    L.ghist1 = take(4 * (size_t)c->max_batch * 2048);
    L.cidx = take(4 * (size_t)c->max_batch * c->max_tokens);
    L.slice_stride = ((size_t)c->max_tokens + 4095) / 4096;
    L.slice_cnt = take(4 * (size_t)c->max_batch * L.slice_stride);
    L.ticket = take(4 * (size_t)c->max_batch);
    const size_t G = c->n_q_heads / c->n_kv_heads;
    size_t rows = (size_t)c->max_chunk * G;
    if (rows > (size_t)kAttSplitRows) rows = kAttSplitRows;
    L.att_elems = (size_t)c->max_batch * c->n_kv_heads * kAttMaxSplits * rows * (c->head_dim + 2);
    // prefill-sized chunks: room for one sequence's key list split kAttPrefillSplits ways
    const size_t big = (size_t)c->n_kv_heads * kAttPrefillSplits * (c->max_chunk * G + 1) * (c->head_dim + 2);
    if ((size_t)c->max_chunk * G > (size_t)kAttSplitRows && big > L.att_elems) L.att_elems = big;
    L.att = take(4 * L.att_elems);
    L.att_count_elems = (size_t)c->max_batch * c->n_kv_heads * ((c->max_chunk * G + 255) / 256);
    L.att_count = take(4 * L.att_count_elems);
    L.status = take(256);
    L.total = off;
    return L;
}

uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);  // NaN
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

esa_status check_common(esa_ctx* ctx, int32_t B) {
    if (!ctx) return ESA_ERR_INVALID_ARG;
    if (B <= 0) return ESA_ERR_INVALID_ARG;
    if (B > ctx->cfg.max_batch) return ESA_ERR_CAPACITY;
    return ESA_OK;
}

// Section 3.1 partition for every sequence of the call.
esa_status build_meta(const esa_ctx* ctx, int B, const int64_t* n_prev, int64_t n_cur, SeqMeta* m,
                      int* max_lM) {
    int mx = 0;
    for (int b = 0; b < B; ++b) {
        const int64_t t = n_prev[b];
        if (t < 0) return ESA_ERR_INVALID_ARG;
        if (t + n_cur > ctx->cfg.max_tokens) return ESA_ERR_CAPACITY;
        const int64_t i_end = t < ctx->cfg.l_init ? t : ctx->cfg.l_init;
        int64_t m_end = t - ctx->cfg.l_local;
        if (m_end < i_end) m_end = i_end;
        m->t[b] = (int)t;
        m->i_end[b] = (int)i_end;
        m->m_end[b] = (int)m_end;
        if (m_end - i_end > mx) mx = (int)(m_end - i_end);
    }
    for (int b = B; b < kMaxBatch; ++b) m->t[b] = m->i_end[b] = m->m_end[b] = 0;
    if (max_lM) *max_lM = mx;
    return ESA_OK;
}

esa_status from_cuda(cudaError_t e) { return e == cudaSuccess ? ESA_OK : ESA_ERR_CUDA; }

// The selection of a step has been enqueued on `st`: the attention call that follows it there may start early.
void arm_attention(esa_ctx* ctx, cudaStream_t st) {
    ctx->sel_armed = true;
    ctx->sel_stream = st;
}

}  // namespace

extern "C" {

const char* esa_status_string(esa_status s) {
    switch (s) {
        case ESA_OK: return "ESA_OK";
        case ESA_ERR_INVALID_ARG: return "ESA_ERR_INVALID_ARG";
        case ESA_ERR_SHAPE: return "ESA_ERR_SHAPE";
        case ESA_ERR_CAPACITY: return "ESA_ERR_CAPACITY";
        case ESA_ERR_CUDA: return "ESA_ERR_CUDA";
        case ESA_ERR_TIMEOUT: return "ESA_ERR_TIMEOUT";
        case ESA_ERR_UNSUPPORTED: return "ESA_ERR_UNSUPPORTED";
        case ESA_ERR_STATE: return "ESA_ERR_STATE";
        case ESA_ERR_INDEX: return "ESA_ERR_INDEX";
    }
    return "ESA_ERR_UNKNOWN";
}

size_t esa_workspace_bytes(const esa_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return make_layout(cfg).total;
}

esa_status esa_create(const esa_config* cfg, esa_ctx** out) {
    if (!out) return ESA_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return ESA_ERR_INVALID_ARG;
    if (!config_ok(cfg)) return ESA_ERR_SHAPE;
    esa_ctx* c = new (std::nothrow) esa_ctx();
    if (!c) return ESA_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->H = cfg->n_q_heads; c->HG = cfg->n_kv_heads; c->d = cfg->head_dim; c->dc = cfg->d_c;
    c->dH = c->H * c->d; c->dG = c->HG * c->d; c->G = c->H / c->HG;
    c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)c->d);
    c->has_w = c->has_bq = c->has_bk = false;
    c->has_wmaps = false;
    c->launches = 0;
    c->last_scored = false;
    c->last_q_rows = 0;
    c->prof_on = false;
    if (cudaGetDevice(&c->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) {
        delete c;
        return ESA_ERR_CUDA;
    }
    Layout L = make_layout(cfg);
    char* base = nullptr;
    if (cudaMalloc(&base, L.total) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return ESA_ERR_CUDA;
    }
    c->ws_bytes = L.total;
    c->base = base;
    c->Wq = reinterpret_cast<__nv_bfloat16*>(base + L.wq);
    c->Wk = reinterpret_cast<__nv_bfloat16*>(base + L.wk);
    c->bq = reinterpret_cast<float*>(base + L.bq);
    c->bk = reinterpret_cast<float*>(base + L.bk);
    c->Qc = reinterpret_cast<__nv_bfloat16*>(base + L.qc);
    c->rkey = reinterpret_cast<uint32_t*>(base + L.rkey);
    c->rkey_heads = reinterpret_cast<uint32_t*>(base + L.rkey_heads);
    c->skey = reinterpret_cast<uint32_t*>(base + L.skey);
    c->pkey = reinterpret_cast<uint32_t*>(base + L.pkey);
    c->ghist0 = reinterpret_cast<uint32_t*>(base + L.ghist0);
    c->ghist1 = reinterpret_cast<uint32_t*>(base + L.ghist1);
    c->cidx = reinterpret_cast<int32_t*>(base + L.cidx);
    c->sel_slice_cnt = reinterpret_cast<int*>(base + L.slice_cnt);
    c->sel_ticket = reinterpret_cast<int*>(base + L.ticket);
    c->sel_slice_stride = (int)L.slice_stride;
    c->last_decode = false;
    c->sel_armed = false;
    c->sel_stream = nullptr;
    c->attend_early = false;
    c->att_part = reinterpret_cast<float*>(base + L.att);
    c->att_part_elems = L.att_elems;
    c->att_count = reinterpret_cast<int*>(base + L.att_count);
    c->att_count_elems = L.att_count_elems;
    c->status = reinterpret_cast<int*>(base + L.status);
    if (cudaMemset(c->status, 0, 256) != cudaSuccess ||
        cudaMemset(c->sel_ticket, 0, 4 * (size_t)cfg->max_batch) != cudaSuccess ||
        cudaMemset(c->ghist1, 0, 4 * (size_t)cfg->max_batch * 2048) != cudaSuccess ||
        cudaMemset(c->att_count, 0, 4 * L.att_count_elems) != cudaSuccess) {
        cudaFree(base);
        delete c;
        return ESA_ERR_CUDA;
    }
    *out = c;
    return ESA_OK;
}

esa_status esa_destroy(esa_ctx* ctx) {
    if (!ctx) return ESA_ERR_INVALID_ARG;
    for (auto& r : ctx->prof_recs) {
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    for (auto ev : ctx->prof_pool) cudaEventDestroy(ev);
    cudaError_t e = cudaFree(ctx->base);
    delete ctx;
    return from_cuda(e);
}

esa_status esa_set_compressors(esa_ctx* ctx, const float* Wq, const float* bq, const float* Wk,
                               const float* bk) {
    if (!ctx || !Wq || !Wk) return ESA_ERR_INVALID_ARG;
    const size_t nq = (size_t)ctx->dc * ctx->dH, nk = (size_t)ctx->dc * ctx->dG;
    std::vector<uint16_t> hq(nq), hk(nk);
    for (size_t i = 0; i < nq; ++i) hq[i] = f32_to_bf16_rne(Wq[i]);
    for (size_t i = 0; i < nk; ++i) hk[i] = f32_to_bf16_rne(Wk[i]);
    if (cudaMemcpy(ctx->Wq, hq.data(), nq * 2, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpy(ctx->Wk, hk.data(), nk * 2, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    ctx->has_bq = bq != nullptr;
    ctx->has_bk = bk != nullptr;
    if (bq && cudaMemcpy(ctx->bq, bq, 4 * ctx->dc, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    if (bk && cudaMemcpy(ctx->bk, bk, 4 * ctx->dc, cudaMemcpyHostToDevice) != cudaSuccess) return ESA_ERR_CUDA;
    ctx->has_wmaps = (ctx->dc == 64 || ctx->dc == 128) && ctx->dH % 128 == 0 && ctx->dG % 128 == 0 &&
                     make_tensor_map_bf16(&ctx->wq_map, ctx->Wq, (uint64_t)ctx->dc, (uint64_t)ctx->dH, (uint32_t)ctx->dc) &&
                     make_tensor_map_bf16(&ctx->wk_map, ctx->Wk, (uint64_t)ctx->dc, (uint64_t)ctx->dG, (uint32_t)ctx->dc);
    ctx->has_w = true;
    return ESA_OK;
}

// ------------------------------------------------------------------ append K/V
esa_status esa_append_kv_async(esa_ctx* ctx, int32_t B, const void* K_new, const void* V_new, int32_t n_new,
                               void* K_cache, void* V_cache, const int64_t* n_prev, void* stream) {
    esa_status s = check_common(ctx, B);
    if (s != ESA_OK) return s;
    if (!K_new || !V_new || !K_cache || !V_cache || !n_prev || n_new < 0) return ESA_ERR_INVALID_ARG;
    RowMap map;
    for (int b = 0; b < B; ++b) {
        if (n_prev[b] < 0) return ESA_ERR_INVALID_ARG;
        if (n_prev[b] + n_new > ctx->cfg.max_tokens) return ESA_ERR_CAPACITY;
        map.row0[b] = (int)n_prev[b];
    }
    if (n_new == 0) return ESA_OK;
    return from_cuda(launch_append_kv(ctx, B, (const __nv_bfloat16*)K_new, (const __nv_bfloat16*)V_new, n_new,
                                      (__nv_bfloat16*)K_cache, (__nv_bfloat16*)V_cache, map,
                                      (cudaStream_t)stream));
}

esa_status esa_append_kv(esa_ctx* ctx, int32_t B, const void* K_new, const void* V_new, int32_t n_new,
                         void* K_cache, void* V_cache, const int64_t* n_prev) {
    esa_status s = esa_append_kv_async(ctx, B, K_new, V_new, n_new, K_cache, V_cache, n_prev, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

// ------------------------------------------------------------- compress keys
esa_status esa_compress_keys_async(esa_ctx* ctx, int32_t B, const void* K_new, int32_t n_new, void* kc_cache,
                                   const int64_t* n_prev, void* stream) {
    esa_status s = check_common(ctx, B);
    if (s != ESA_OK) return s;
    if (!K_new || !kc_cache || !n_prev || n_new < 0) return ESA_ERR_INVALID_ARG;
    if (!ctx->has_w) return ESA_ERR_STATE;
    const int cap = ctx->cfg.max_chunk > kCompressMaxRows ? ctx->cfg.max_chunk : kCompressMaxRows;
    if (n_new > cap) return ESA_ERR_CAPACITY;
    RowMap map;
    for (int b = 0; b < B; ++b) {
        if (n_prev[b] < 0) return ESA_ERR_INVALID_ARG;
        if (n_prev[b] + n_new > ctx->cfg.max_tokens) return ESA_ERR_CAPACITY;
        map.row0[b] = (int)n_prev[b];
    }
    if (n_new == 0) return ESA_OK;
    if (B * n_new <= kCompressGemvRows) {
        cudaError_t e = launch_compress_gemv(ctx, (const __nv_bfloat16*)K_new, B, n_new, ctx->dG, ctx->Wk,
                                             ctx->has_bk ? ctx->bk : nullptr, (__nv_bfloat16*)kc_cache,
                                             ctx->cfg.max_tokens, map, nullptr, 0, nullptr, 0, (cudaStream_t)stream);
        if (e != cudaErrorNotSupported) return from_cuda(e);
        cudaGetLastError();
    }
    if (ctx->has_wmaps) {
        cudaError_t e = launch_compress_tc(ctx, (const __nv_bfloat16*)K_new, B, n_new, ctx->dG, &ctx->wk_map,
                                           ctx->has_bk ? ctx->bk : nullptr, (__nv_bfloat16*)kc_cache,
                                           ctx->cfg.max_tokens, map, nullptr, 0, (cudaStream_t)stream, true);
        if (e != cudaErrorNotSupported) return from_cuda(e);
        cudaGetLastError();
    }
    return from_cuda(launch_compress(ctx, (const __nv_bfloat16*)K_new, B, n_new, ctx->dG, ctx->Wk,
                                     ctx->has_bk ? ctx->bk : nullptr, (__nv_bfloat16*)kc_cache,
                                     ctx->cfg.max_tokens, map, (cudaStream_t)stream));
}

esa_status esa_compress_keys(esa_ctx* ctx, int32_t B, const void* K_new, int32_t n_new, void* kc_cache,
                             const int64_t* n_prev) {
    esa_status s = esa_compress_keys_async(ctx, B, K_new, n_new, kc_cache, n_prev, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

// -------------------------------------------------------------------- select
esa_status esa_select_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* kc_cache,
                            const int64_t* n_prev, int32_t* idx_out, int32_t* n_sel_out, void* stream) {
    esa_status s = check_common(ctx, B);
    if (s != ESA_OK) return s;
    if (!Q_cur || !kc_cache || !n_prev || !idx_out || !n_sel_out || l_C <= 0) return ESA_ERR_INVALID_ARG;
    if (l_C > ctx->cfg.max_chunk) return ESA_ERR_CAPACITY;
    if (!ctx->has_w) return ESA_ERR_STATE;
    SeqMeta meta;
    int max_lM = 0;
    s = build_meta(ctx, B, n_prev, l_C, &meta, &max_lM);
    if (s != ESA_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    bool any_small = false, any_large = false;
    for (int b = 0; b < B; ++b) {
        int lM = meta.m_end[b] - meta.i_end[b];
        ctx->last_lM[b] = lM;
        if (lM > ctx->cfg.top_k) any_large = true; else any_small = true;
    }
    ctx->last_scored = any_large;
    ctx->last_q_rows = any_large ? (int64_t)B * l_C : 0;
    cudaError_t e = cudaSuccess;
    if (any_small) {
        e = launch_select_all(ctx, B, meta, idx_out, n_sel_out, st);
        if (e != cudaSuccess) return ESA_ERR_CUDA;
    }
    if (!any_large) {
        arm_attention(ctx, st);
        return ESA_OK;
    }
    // q' = f_q(q) (Eq. 5)
    RowMap zero;
    for (int b = 0; b < kMaxBatch; ++b) zero.row0[b] = 0;
    e = cudaErrorNotSupported;
    bool rkey_cleared = false, ghist_cleared = false;
    if (B * l_C <= kCompressGemvRows) {
        // (with one query per sequence the scoring kernel also accumulates first-digit histograms: cleared here too)
        e = launch_compress_gemv(ctx, (const __nv_bfloat16*)Q_cur, B, l_C, ctx->dH, ctx->Wq,
                                 ctx->has_bq ? ctx->bq : nullptr, ctx->Qc, l_C, zero, ctx->rkey, B * l_C,
                                 l_C == 1 ? ctx->ghist0 : nullptr, B * 2048, st);
        rkey_cleared = e == cudaSuccess;
        ghist_cleared = rkey_cleared && l_C == 1;
    }
    if (e == cudaErrorNotSupported && ctx->has_wmaps) {
        // the compression kernel also clears the row-maximum words that the scoring pass accumulates into
        e = launch_compress_tc(ctx, (const __nv_bfloat16*)Q_cur, B, l_C, ctx->dH, &ctx->wq_map,
                               ctx->has_bq ? ctx->bq : nullptr, ctx->Qc, l_C, zero, ctx->rkey, B * l_C, st);
        rkey_cleared = e == cudaSuccess;
    }
    if (e == cudaErrorNotSupported) {
        cudaGetLastError();
        e = launch_compress(ctx, (const __nv_bfloat16*)Q_cur, B, l_C, ctx->dH, ctx->Wq,
                            ctx->has_bq ? ctx->bq : nullptr, ctx->Qc, l_C, zero, st);
    }
    if (e != cudaSuccess) return ESA_ERR_CUDA;
    // sequences that select everything need no scores: give them an empty middle part
    SeqMeta smeta = meta;
    for (int b = 0; b < B; ++b)
        if (meta.m_end[b] - meta.i_end[b] <= ctx->cfg.top_k) smeta.m_end[b] = smeta.i_end[b];
    ctx->last_decode = l_C == 1;
    bool pooled_ready = false;
    e = launch_score(ctx, B, l_C, (const __nv_bfloat16*)kc_cache, smeta, max_lM, rkey_cleared, ghist_cleared, st,
                     &pooled_ready);
    if (e != cudaSuccess) return ESA_ERR_CUDA;
    e = launch_select(ctx, B, l_C == 1, smeta, max_lM, pooled_ready, idx_out, n_sel_out, st);
    if (e == cudaSuccess) arm_attention(ctx, st);
    return from_cuda(e);
}

esa_status esa_select_full_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_cache,
                                 const int64_t* n_prev, int32_t mode, int32_t* idx_out, int32_t* n_sel_out, void* stream) {
    esa_status s = check_common(ctx, B);
    if (s != ESA_OK) return s;
    if (!Q_cur || !K_cache || !n_prev || !idx_out || !n_sel_out || l_C <= 0) return ESA_ERR_INVALID_ARG;
    if (mode != ESA_SCORE_UNIFORM && mode != ESA_SCORE_PER_HEAD) return ESA_ERR_INVALID_ARG;
    if (l_C > ctx->cfg.max_chunk) return ESA_ERR_CAPACITY;
    SeqMeta meta;
    int max_lM = 0;
    s = build_meta(ctx, B, n_prev, l_C, &meta, &max_lM);
    if (s != ESA_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    bool any_small = false, any_large = false;
    for (int b = 0; b < B; ++b) {
        int lM = meta.m_end[b] - meta.i_end[b];
        ctx->last_lM[b] = lM;
        if (lM > ctx->cfg.top_k) any_large = true; else any_small = true;
    }
    ctx->last_scored = any_large;
    ctx->last_q_rows = 0;
    if (any_small && launch_select_all(ctx, B, meta, idx_out, n_sel_out, st) != cudaSuccess) return ESA_ERR_CUDA;
    if (!any_large) {
        arm_attention(ctx, st);
        return ESA_OK;
    }
    SeqMeta smeta = meta;
    for (int b = 0; b < B; ++b)
        if (meta.m_end[b] - meta.i_end[b] <= ctx->cfg.top_k) smeta.m_end[b] = smeta.i_end[b];
    ctx->last_decode = false;
    cudaError_t e = launch_score_full(ctx, B, l_C, (const __nv_bfloat16*)Q_cur, (const __nv_bfloat16*)K_cache, smeta, max_lM,
                                      mode == ESA_SCORE_PER_HEAD, st);
    if (e != cudaSuccess) return ESA_ERR_CUDA;
    e = launch_select(ctx, B, false, smeta, max_lM, false, idx_out, n_sel_out, st);
    if (e == cudaSuccess) arm_attention(ctx, st);
    return from_cuda(e);
}

esa_status esa_select_full(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_cache,
                           const int64_t* n_prev, int32_t mode, int32_t* idx_out, int32_t* n_sel_out) {
    esa_status s = esa_select_full_async(ctx, B, Q_cur, l_C, K_cache, n_prev, mode, idx_out, n_sel_out, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

esa_status esa_select(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* kc_cache,
                      const int64_t* n_prev, int32_t* idx_out, int32_t* n_sel_out) {
    esa_status s = esa_select_async(ctx, B, Q_cur, l_C, kc_cache, n_prev, idx_out, n_sel_out, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

// -------------------------------------------------------------------- attend
esa_status esa_attend_two_position_async(esa_ctx* ctx, int32_t B, const void* Q_cur, const void* Q_far, int32_t l_C,
                                         const void* K_cache, const void* K_far_cache, const void* V_cache,
                                         const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel, void* O,
                                         void* stream) {
    esa_status s = check_common(ctx, B);
    if (s != ESA_OK) return s;
    if (!Q_cur || !K_cache || !V_cache || !n_prev || !idx || !n_sel || !O || l_C <= 0) return ESA_ERR_INVALID_ARG;
    if (l_C > ctx->cfg.max_chunk) return ESA_ERR_CAPACITY;
    SeqMeta meta;
    s = build_meta(ctx, B, n_prev, l_C, &meta, nullptr);
    if (s != ESA_OK) return s;
    // a call that follows the selection of its step on the same stream may attend the older rows early
    ctx->attend_early = ctx->sel_armed && ctx->sel_stream == (cudaStream_t)stream;
    ctx->sel_armed = false;
    cudaError_t e = launch_attend(ctx, B, l_C, (const __nv_bfloat16*)Q_cur, (const __nv_bfloat16*)Q_far,
                                  (const __nv_bfloat16*)K_cache, (const __nv_bfloat16*)K_far_cache,
                                  (const __nv_bfloat16*)V_cache, meta, idx, n_sel, (__nv_bfloat16*)O,
                                  (cudaStream_t)stream);
    ctx->attend_early = false;
    return from_cuda(e);
}

esa_status esa_attend_two_position(esa_ctx* ctx, int32_t B, const void* Q_cur, const void* Q_far, int32_t l_C,
                                   const void* K_cache, const void* K_far_cache, const void* V_cache,
                                   const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel, void* O) {
    esa_status s = esa_attend_two_position_async(ctx, B, Q_cur, Q_far, l_C, K_cache, K_far_cache, V_cache, n_prev, idx,
                                                 n_sel, O, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

esa_status esa_attend_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_cache,
                            const void* V_cache, const int64_t* n_prev, const int32_t* idx,
                            const int32_t* n_sel, void* O, void* stream) {
    return esa_attend_two_position_async(ctx, B, Q_cur, nullptr, l_C, K_cache, nullptr, V_cache, n_prev, idx, n_sel, O,
                                         stream);
}

esa_status esa_attend(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_cache,
                      const void* V_cache, const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel,
                      void* O) {
    esa_status s = esa_attend_async(ctx, B, Q_cur, l_C, K_cache, V_cache, n_prev, idx, n_sel, O, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

// ------------------------------------------------------- host-resident K/V
esa_status esa_attend_host_kv_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_host,
                                    const void* V_host, const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel,
                                    void* K_stage, void* V_stage, int64_t stage_rows, void* O, void* stream) {
    esa_status s = check_common(ctx, B);
    if (s != ESA_OK) return s;
    if (!Q_cur || !K_host || !V_host || !n_prev || !idx || !n_sel || !K_stage || !V_stage || !O || l_C <= 0)
        return ESA_ERR_INVALID_ARG;
    if (l_C > ctx->cfg.max_chunk) return ESA_ERR_CAPACITY;
    SeqMeta meta;
    s = build_meta(ctx, B, n_prev, l_C, &meta, nullptr);
    if (s != ESA_OK) return s;
    // rows of the attended list per sequence (the selection may hold fewer than top_k: the upper bound sizes the stage)
    for (int b = 0; b < B; ++b) {
        const int lM = meta.m_end[b] - meta.i_end[b];
        const int64_t n_att = (int64_t)meta.i_end[b] + (lM < ctx->cfg.top_k ? lM : ctx->cfg.top_k) + (meta.t[b] - meta.m_end[b]) + l_C;
        if (n_att > stage_rows) return ESA_ERR_CAPACITY;
    }
    if (stage_rows >= (int64_t(1) << 31)) return ESA_ERR_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    ctx->sel_armed = false;       // (the staged list is written by the gather kernel just ahead: never attended early)
    if (launch_gather_kv(ctx, B, l_C, K_host, V_host, meta, idx, n_sel, K_stage, V_stage, stage_rows, st) != cudaSuccess)
        return ESA_ERR_CUDA;
    // The staged rows are the attended list itself: the attention kernels run on the same partition with the
    // identity as the map from list positions to cache rows.
    return from_cuda(launch_attend(ctx, B, l_C, (const __nv_bfloat16*)Q_cur, nullptr, (const __nv_bfloat16*)K_stage, nullptr,
                                   (const __nv_bfloat16*)V_stage, meta, idx, n_sel, (__nv_bfloat16*)O, st, stage_rows, true));
}

esa_status esa_attend_host_kv(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_host,
                              const void* V_host, const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel,
                              void* K_stage, void* V_stage, int64_t stage_rows, void* O) {
    esa_status s = esa_attend_host_kv_async(ctx, B, Q_cur, l_C, K_host, V_host, n_prev, idx, n_sel, K_stage, V_stage,
                                            stage_rows, O, nullptr);
    if (s != ESA_OK) return s;
    return from_cuda(cudaStreamSynchronize(nullptr));
}

// --------------------------------------------------------------- diagnostics
esa_status esa_read_pooled_scores(esa_ctx* ctx, int32_t b, float* dst_host, int64_t n, void* stream) {
    if (!ctx || !dst_host || b < 0 || b >= ctx->cfg.max_batch || n < 0) return ESA_ERR_INVALID_ARG;
    if (!ctx->last_scored || ctx->last_lM[b] <= ctx->cfg.top_k) return ESA_ERR_STATE;
    if (n > ctx->last_lM[b]) return ESA_ERR_CAPACITY;
    if (n == 0) return ESA_OK;
    cudaStream_t st = (cudaStream_t)stream;
    // the candidate-key buffer of this sequence is free again after the selection: stage there
    float* tmp = reinterpret_cast<float*>(ctx->skey + (int64_t)b * ctx->cfg.max_tokens);
    if (launch_read_pooled(ctx, b, tmp, n, st) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaMemcpyAsync(dst_host, tmp, 4 * (size_t)n, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ESA_ERR_CUDA;
    return from_cuda(cudaStreamSynchronize(st));
}

esa_status esa_read_compressed_queries(esa_ctx* ctx, void* dst_host, int64_t n_rows, void* stream) {
    if (!ctx || !dst_host || n_rows < 0) return ESA_ERR_INVALID_ARG;
    if (!ctx->last_scored || ctx->last_q_rows == 0) return ESA_ERR_STATE;
    if (n_rows > ctx->last_q_rows) return ESA_ERR_CAPACITY;
    if (n_rows == 0) return ESA_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(dst_host, ctx->Qc, 2 * (size_t)n_rows * ctx->dc, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ESA_ERR_CUDA;
    return from_cuda(cudaStreamSynchronize(st));
}

esa_status esa_debug_wait_timeout(esa_ctx* ctx, int64_t limit_cycles, void* stream) {
    if (!ctx || limit_cycles < 1 || limit_cycles > 2000000000LL) return ESA_ERR_INVALID_ARG;
    return from_cuda(launch_debug_wait(ctx, limit_cycles, (cudaStream_t)stream));
}

int32_t esa_kernel_class_count(void) { return KC_COUNT; }

const char* esa_kernel_class_name(int32_t cls) {
    static const char* names[KC_COUNT] = {
        "compress_tc_kernel", "compress_gemv_kernel", "compress_kernel", "append_kv_kernel", "score_tc_kernel<.,1>",
        "score_tc_kernel<.,2>", "score_pass_kernel<.,1>+<.,2>", "score_decode_kernel", "score_full_kernel<.,1>+<.,2>",
        "pool_hist_kernel",
        "select_topk_kernel", "select_all_kernel", "attend_tc_kernel", "attend_decode_kernel", "attend_kernel",
        "attend_merge_kernel", "gather_kv_kernel"};
    return cls >= 0 && cls < KC_COUNT ? names[cls] : "";
}

esa_status esa_set_profiling(esa_ctx* ctx, int32_t on) {
    if (!ctx) return ESA_ERR_INVALID_ARG;
    ctx->prof_on = on != 0;
    return ESA_OK;
}

esa_status esa_read_profile(esa_ctx* ctx, int32_t n_classes, int64_t* launches, double* total_ms) {
    if (!ctx || !launches || !total_ms || n_classes < KC_COUNT) return ESA_ERR_INVALID_ARG;
    for (int i = 0; i < n_classes; ++i) {
        launches[i] = 0;
        total_ms[i] = 0.0;
    }
    esa_status result = ESA_OK;
    for (auto& r : ctx->prof_recs) {
        float ms = 0.f;
        if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) {
            cudaGetLastError();
            result = ESA_ERR_CUDA;
        } else {
            launches[r.cls] += 1;
            total_ms[r.cls] += ms;
        }
        ctx->prof_pool.push_back(r.a);
        ctx->prof_pool.push_back(r.b);
    }
    ctx->prof_recs.clear();
    return result;
}

int64_t esa_launch_count(const esa_ctx* ctx) { return ctx ? ctx->launches : -1; }

esa_status esa_last_device_status(esa_ctx* ctx, void* stream) {
    if (!ctx) return ESA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int h = 0;
    if (cudaMemcpyAsync(&h, ctx->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ESA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ESA_ERR_CUDA;
    if (h != 0) {
        if (cudaMemsetAsync(ctx->status, 0, sizeof(int), st) != cudaSuccess) return ESA_ERR_CUDA;
        // a kernel that gave up may have left arrival counters of the in-kernel merges behind
        if (cudaMemsetAsync(ctx->att_count, 0, sizeof(int) * ctx->att_count_elems, st) != cudaSuccess) return ESA_ERR_CUDA;
        if (cudaMemsetAsync(ctx->sel_ticket, 0, sizeof(int) * ctx->cfg.max_batch, st) != cudaSuccess) return ESA_ERR_CUDA;
        if (cudaMemsetAsync(ctx->ghist1, 0, sizeof(uint32_t) * ctx->cfg.max_batch * 2048, st) != cudaSuccess) return ESA_ERR_CUDA;
        return (esa_status)h;
    }
    return ESA_OK;
}

}  // extern "C"
