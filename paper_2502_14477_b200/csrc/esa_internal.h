// Host-side declarations shared by the translation units of the ESA library.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/esa.h"
#include "esa_common.cuh"

namespace esa {

// Launch with the programmatic-serialization attribute (the kernel must call pdl_wait() before it
// touches global memory).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kAttMaxSplits = 64;     // split-KV factor of the attention kernel (small chunks)
constexpr int kAttSplitRows = 64;     // split-KV is used only when l_C * (H/H_G) <= this
constexpr int kAttPrefillSplits = 4; // largest split of a prefill-sized chunk's key list
constexpr int kCompressGemvRows = 16;   // at most this many input rows (B * n_new): compression runs as a GEMV
constexpr int kCompressMaxRows = 4096;

// Destination rows of a compression: row i of sequence b goes to
// dst[(b * seq_stride + row0[b] + i) * d_c ...].
struct RowMap {
    int row0[kMaxBatch];
};

// Kernel classes of the per-kernel timing facility (esa_set_profiling / esa_read_profile).
enum KernelClass {
    KC_COMPRESS_TC = 0, KC_COMPRESS_GEMV, KC_COMPRESS_MMA, KC_APPEND_KV, KC_SCORE_PASS1, KC_SCORE_PASS2, KC_SCORE_MMA,
    KC_SCORE_DECODE, KC_SCORE_FULL, KC_POOL_HIST, KC_SELECT_TOPK, KC_SELECT_ALL, KC_ATTEND_TC, KC_ATTEND_DECODE, KC_ATTEND_SMALL,
    KC_ATTEND_MERGE, KC_GATHER_KV, KC_COUNT
};
struct ProfRec {
    int cls;
    cudaEvent_t a, b;
};

}  // namespace esa

struct esa_ctx {
    esa_config cfg;
    int device;
    void* base;          // the single device allocation every pointer below points into
    int num_sms;
    int H, HG, d, dc, dH, dG, G;
    float scale;
    bool has_w, has_bq, has_bk;
    __nv_bfloat16* Wq;   // [dc, dH]
    __nv_bfloat16* Wk;   // [dc, dG]
    CUtensorMap wq_map, wk_map;   // TMA descriptors of Wq / Wk (valid when has_wmaps)
    bool has_wmaps;
    float* bq;           // [dc]
    float* bk;           // [dc]
    __nv_bfloat16* Qc;   // [max_batch * max_chunk, dc]
    uint32_t* rkey;      // [max_batch * max_chunk] ordered keys of the row maxima r_c
    uint32_t* rkey_heads;  // [max_batch, H, max_chunk] row maxima of the full-dimension / per-head scoring variants
    uint32_t* skey;      // [max_batch, max_tokens] unpooled aggregated scores (ordered keys) of the scoring paths that do not pool;
                         // afterwards the selection's candidate keys
    uint32_t* pkey;      // [max_batch, max_tokens] pooled scores s' as ordered keys (l_C = 1: of the pooled raw scores, r not yet subtracted)
    uint32_t* ghist0;    // [max_batch, 2048] histograms of pkey's top 11 bits (first radix digit)
    uint32_t* ghist1;    // [max_batch, 2048] second-digit histograms of the selection kernel; 0 between launches
    int32_t* cidx;       // [max_batch, max_tokens] positions of the selection's candidates
    int* sel_slice_cnt;  // [max_batch, sel_slice_stride] candidates per slice of the selection kernel (sized for 4096-token slices, the kernel uses larger ones)
    int* sel_ticket;     // [max_batch] arrival tickets of the selection kernel; 0 between launches
    int sel_slice_stride;
    bool last_decode;    // the last selection ran with l_C = 1 (pkey holds raw pooled scores)
    // The attention kernels may read cache rows older than the chunk ahead of their wait for the preceding kernel
    // only when the work ahead of them in the stream is known not to write such rows: a selection enqueued through
    // this context arms the next attention call on the same stream (the caller's side of it: nothing enqueued
    // between the two calls writes cache rows older than the chunk).
    bool sel_armed;
    cudaStream_t sel_stream;
    bool attend_early;   // set around the launch of an armed attention call
    float* att_part;     // split-KV partial outputs + (m, l)
    size_t att_part_elems;
    int* att_count;      // arrival counters of the split prefill attention, one per (sequence, kv head, row tile); 0 between launches
    size_t att_count_elems;
    int* status;         // device status word
    int64_t launches;
    int last_lM[esa::kMaxBatch];
    bool last_scored;
    int64_t last_q_rows;  // rows of q' left in Qc by the last selection that scored
    size_t ws_bytes;
    bool prof_on;                          // bracket every kernel launch with CUDA events
    std::vector<esa::ProfRec> prof_recs;   // launches recorded since the last esa_read_profile
    std::vector<cudaEvent_t> prof_pool;    // events free for reuse
};

namespace esa {

// While profiling is on, records a CUDA event on the launching stream before and after the kernel(s)
// launched during its lifetime (class `cls`).  An event between two kernels keeps the second from being
// set up under the first one's tail, so profiled calls run without the dependent-launch overlap.
struct ProfScope {
    esa_ctx* c;
    cudaStream_t st;
    cudaEvent_t b;
    bool on;
    ProfScope(esa_ctx* ctx, int cls, cudaStream_t stream) : c(ctx), st(stream), b(nullptr), on(ctx->prof_on) {
        if (!on) return;
        cudaEvent_t ev[2] = {nullptr, nullptr};
        for (int i = 0; i < 2; ++i) {
            if (!c->prof_pool.empty()) {
                ev[i] = c->prof_pool.back();
                c->prof_pool.pop_back();
            } else if (cudaEventCreate(&ev[i]) != cudaSuccess) {
                on = false;
                return;
            }
        }
        cudaEventRecord(ev[0], st);
        b = ev[1];
        c->prof_recs.push_back(ProfRec{cls, ev[0], ev[1]});
    }
    ~ProfScope() {
        if (on) cudaEventRecord(b, st);
    }
};

// Y[dst rows] = bf16( X[rows, d_in] . W[dc, d_in]^T + bias ), fp32 accumulation, split-K.
cudaError_t launch_compress(esa_ctx* ctx, const __nv_bfloat16* X, int B, int rows_per_seq, int d_in,
                            const __nv_bfloat16* W, const float* bias, __nv_bfloat16* dst,
                            int64_t dst_seq_stride, const RowMap& map, cudaStream_t st);

// Eq. 6 + Eq. 4: fills ctx->skey (and ctx->rkey) for the middle tokens of every sequence.
// l_C = 1: fills ctx->pkey (pooled raw scores), ctx->ghist0 and ctx->rkey instead.
// rkey_cleared / ghist_cleared: the caller's compression kernel has already zeroed ctx->rkey / ctx->ghist0 for this call.
// *pooled_ready: ctx->pkey and ctx->ghist0 hold the pooled keys and their first-digit histogram; otherwise
// ctx->skey holds unpooled keys and ctx->ghist0 is zero.
cudaError_t launch_score(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache,
                         const SeqMeta& meta, int max_lM, bool rkey_cleared, bool ghist_cleared, cudaStream_t st,
                         bool* pooled_ready);

// The same for chunks of >= 64 queries and d' in {64, 128} on tcgen05 with TMA-fed tiles; expects
// ctx->rkey zeroed (pass 1 clears what pass 2 accumulates into).  cudaErrorNotSupported when the shape is not covered.
cudaError_t launch_score_tc(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache,
                            const SeqMeta& meta, int max_lM, cudaStream_t st, bool* pooled_ready);

// Eq. 8 (unless pooled_ready) + Eq. 2 -> idx_out / n_sel_out.  mapped: ctx->pkey holds the pooled RAW scores of a
// single query per sequence and ctx->rkey[b] its maximum (the decode scoring kernel's output).
cudaError_t launch_select(esa_ctx* ctx, int B, bool mapped, const SeqMeta& meta, int max_lM, bool pooled_ready,
                          int32_t* idx_out, int32_t* n_sel_out, cudaStream_t st);

// Eq. 3 + Eq. 4 on the uncompressed queries and keys (per_head: the per-head vote of Section 4.3): unpooled keys to
// ctx->skey, ctx->ghist0 zeroed.
cudaError_t launch_score_full(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* K, const SeqMeta& meta,
                              int max_lM, bool per_head, cudaStream_t st);

// idx_out[b, 0..l_M) = i_end + 0..l_M-1, n_sel_out[b] = l_M for sequences with l_M <= top_k
// (only_small = 1) or all sequences (only_small = 0).
cudaError_t launch_select_all(esa_ctx* ctx, int B, const SeqMeta& meta, int32_t* idx_out,
                              int32_t* n_sel_out, cudaStream_t st);

// Qg / Kg: queries and key cache used against I and M_k (two-position attention, Section 3.2); null = Q / K.
// cache_rows: rows per sequence of the K/V caches handed in (0 = the configuration's max_tokens).
// staged: the caches hold the attended list itself, row j = list entry j (host-resident K/V, staged by launch_gather_kv).
cudaError_t launch_attend(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* Qg,
                          const __nv_bfloat16* K, const __nv_bfloat16* Kg, const __nv_bfloat16* V, const SeqMeta& meta,
                          const int32_t* idx, const int32_t* n_sel, __nv_bfloat16* O, cudaStream_t st,
                          int64_t cache_rows = 0, bool staged = false);

// Host-resident K/V: copies the rows of the attended list, in list order, into device staging caches.
cudaError_t launch_gather_kv(esa_ctx* ctx, int B, int l_C, const void* K_host, const void* V_host, const SeqMeta& meta,
                             const int32_t* idx, const int32_t* n_sel, void* K_stage, void* V_stage, int64_t stage_rows,
                             cudaStream_t st);

// Prefill-sized chunks (l_C * H/H_G > kAttSplitRows) on tcgen05; *nsplit_out reports the number of
// key-list splits (their partials pass through ctx->att_part and are merged inside the kernel).
// Qg / Kg non-null: two-position attention (both given then).
cudaError_t launch_attend_tc(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* Qg,
                             const __nv_bfloat16* K, const __nv_bfloat16* Kg, const __nv_bfloat16* V, const SeqMeta& meta,
                             const int32_t* idx, const int32_t* n_sel, __nv_bfloat16* O,
                             int n_att_max, cudaStream_t st, int* nsplit_out, int64_t cache_rows = 0, bool staged = false);

// TMA descriptor of a row-major bf16 matrix [rows, cols] (cols a multiple of 64), read in boxes of
// box_rows x 64 columns with the 128-byte swizzle.  False when the driver entry point is missing
// or refuses the shape.
bool make_tensor_map_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// TMA descriptor of the query tensor [n_queries, H, D] for the attention kernel (group size G must
// divide 128).
bool make_tensor_map_q(CUtensorMap* map, const void* base, uint64_t n_queries, int H, int D, int G);

// Eq. 5 on tcgen05 for d' in {64, 128} and d_in a multiple of 128.  X is [rows, d_in] contiguous.
// cudaErrorNotSupported when the shape is not covered (the caller then uses the mma.sync kernel).
// Compression of a handful of rows (B * rows_per_seq <= kCompressGemvRows) as a GEMV; optionally clears
// zero_count words at zero_words (one CTA) and zero2_count words at zero2_words (spread over the grid).  cudaErrorNotSupported when the shape is not covered.
cudaError_t launch_compress_gemv(esa_ctx* ctx, const __nv_bfloat16* X, int B, int rows_per_seq, int d_in,
                                 const __nv_bfloat16* W, const float* bias, __nv_bfloat16* dst,
                                 int64_t dst_seq_stride, const RowMap& map, uint32_t* zero_words, int zero_count,
                                 uint32_t* zero2_words, int zero2_count, cudaStream_t st);
// small_grid: the result is not needed at once (key compression: its rows enter M only l_L tokens later, and callers
// run it on a side stream), so the grid is kept to an eighth of the SMs instead of as many CTAs as shorten the call.
cudaError_t launch_compress_tc(esa_ctx* ctx, const __nv_bfloat16* X, int B, int rows_per_seq, int d_in,
                               const CUtensorMap* wmap, const float* bias, __nv_bfloat16* dst,
                               int64_t dst_seq_stride, const RowMap& map, uint32_t* zero_words, int zero_count,
                               cudaStream_t st, bool small_grid = false);

// True when launch_score takes the tcgen05 path for this call.
inline bool score_uses_tc(const esa_ctx* ctx, int B, int l_C) {
    return l_C >= 64 && (ctx->dc == 64 || ctx->dc == 128) &&
           (int64_t)B * ctx->cfg.max_tokens < (int64_t(1) << 31);
}

cudaError_t launch_append_kv(esa_ctx* ctx, int B, const __nv_bfloat16* K_new,
                             const __nv_bfloat16* V_new, int n_new, __nv_bfloat16* K_cache,
                             __nv_bfloat16* V_cache, const RowMap& map, cudaStream_t st);

cudaError_t launch_read_pooled(esa_ctx* ctx, int b, float* dst_dev, int64_t n, cudaStream_t st);

// One thread waits on a barrier nobody completes, for at most limit_cycles: exercises the give-up path.
cudaError_t launch_debug_wait(esa_ctx* ctx, int64_t limit_cycles, cudaStream_t st);

}  // namespace esa
