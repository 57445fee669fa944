// Eq. 6 + Eq. 4: importance scores of the middle tokens against the current chunk.
//
//   S[c, m] = q'_c . k'_m                     (Eq. 6, bf16 products, fp32 accumulation)
//   r_c     = max_m S[c, m]
//   s_m     = max_c ( S[c, m] - r_c )         (Eq. 4)
//
// S is never written to memory.  Eq. 4 needs every r_c before any s_m, so the
// contraction runs twice over the compressed keys (they are only d' wide): pass 1
// keeps the column maxima r_c, pass 2 recomputes S and folds max_c(S - r_c) into its
// epilogue.  Both passes put the keys on the M side of the MMA and the queries on the
// N side and issue the same instruction sequence, so pass 2 reproduces pass 1's S bit
// for bit and S - r_c <= 0 with equality at each query's arg-max.
//
// For a single query (decode) the contraction is a matrix-vector product bound by the
// read of the compressed keys; it runs on CUDA cores and stores the raw S, and the
// subtraction of r_0 is applied when the selection kernel reads the scores.
#include "esa_internal.h"

namespace esa {

constexpr int SC_BM = 128;      // keys per tile (8 warps x 16)
constexpr int SC_BN = 128;      // queries per CTA
constexpr int SC_THREADS = 256;
constexpr int SC_STAGES = 3;

struct ScoreParams {
    const __nv_bfloat16* kc;    // [B, max_tokens, DC]
    const __nv_bfloat16* qc;    // [B, l_C, DC]
    uint32_t* rkey;             // [B, l_C]
    uint32_t* skey;             // [B, max_tokens] (index = m - i_end)
    int64_t max_tokens;
    int l_C;
    SeqMeta meta;
};

template <int DC, int PASS>
__global__ void __launch_bounds__(SC_THREADS)
score_pass_kernel(ScoreParams p) {
    constexpr int CH = DC / 8;
    extern __shared__ uint4 smem[];
    uint4* sQ = smem;                                  // [SC_BN][CH]
    uint4* sK = smem + SC_BN * CH;                     // SC_STAGES x [SC_BM][CH]
    float* sR = reinterpret_cast<float*>(sK + SC_STAGES * SC_BM * CH);  // [8][SC_BN] (pass 1) / [SC_BN] (pass 2)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.z;
    const int q0 = blockIdx.y * SC_BN;
    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int n_tiles = (l_M + SC_BM - 1) / SC_BM;
    if ((int)blockIdx.x >= n_tiles) return;
    const __nv_bfloat16* kc = p.kc + ((int64_t)b * p.max_tokens + i_end) * DC;
    const __nv_bfloat16* qc = p.qc + (int64_t)b * p.l_C * DC;

    // queries of this CTA -> smem (rows past l_C are zero)
    for (int i = tid; i < SC_BN * CH; i += SC_THREADS) {
        int r = i / CH, c = i % CH;
        bool ok = q0 + r < p.l_C;
        cp_async16(&sQ[swz<CH>(r, c)], qc + (int64_t)(ok ? q0 + r : 0) * DC + c * 8, ok ? 16 : 0);
    }
    auto load_tile = [&](int st, int tile) {
        const int m0 = tile * SC_BM;
        uint4* dst = sK + st * SC_BM * CH;
        for (int i = tid; i < SC_BM * CH; i += SC_THREADS) {
            int r = i / CH, c = i % CH;
            bool ok = m0 + r < l_M;
            cp_async16(&dst[swz<CH>(r, c)], kc + (int64_t)(ok ? m0 + r : 0) * DC + c * 8, ok ? 16 : 0);
        }
    };

    // r_c of this thread's query columns (pass 2) / running column maxima (pass 1)
    float colv[SC_BN / 8][2];
    if (PASS == 2) {
        for (int i = tid; i < SC_BN; i += SC_THREADS)
            sR[i] = (q0 + i < p.l_C) ? key_to_f32(p.rkey[(int64_t)b * p.l_C + q0 + i]) : INFINITY;
    }

    int tile = blockIdx.x;
    int issued = 0;
    for (int s = 0; s < SC_STAGES - 1; ++s) {
        if (tile + s * (int)gridDim.x < n_tiles) load_tile(s, tile + s * gridDim.x);
        cp_async_commit();
        ++issued;
    }
    __syncthreads();
#pragma unroll
    for (int nb = 0; nb < SC_BN / 8; ++nb) {
        if (PASS == 2) {
            colv[nb][0] = sR[nb * 8 + (lane & 3) * 2];
            colv[nb][1] = sR[nb * 8 + (lane & 3) * 2 + 1];
        } else {
            colv[nb][0] = colv[nb][1] = -INFINITY;
        }
    }

    int it = 0;
    for (; tile < n_tiles; tile += gridDim.x, ++it) {
        // prefetch the tile SC_STAGES-1 ahead, then wait for the current one
        {
            int nt = tile + (SC_STAGES - 1) * gridDim.x;
            if (nt < n_tiles) load_tile((it + SC_STAGES - 1) % SC_STAGES, nt);
            cp_async_commit();
        }
        cp_async_wait<SC_STAGES - 1>();
        __syncthreads();
        const uint4* tk = sK + (it % SC_STAGES) * SC_BM * CH;

        float acc[SC_BN / 8][4];
#pragma unroll
        for (int i = 0; i < SC_BN / 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll
        for (int ks = 0; ks < DC / 16; ++ks) {
            uint32_t a[4];
            load_a_frag<CH>(a, tk, warp * 16, ks * 2, lane);
#pragma unroll
            for (int nb = 0; nb < SC_BN / 16; ++nb) {
                uint32_t bq[4];
                load_b_frag_nk<CH>(bq, sQ, nb * 16, ks * 2, lane);
                mma_bf16_16816(acc[2 * nb], a, bq[0], bq[1]);
                mma_bf16_16816(acc[2 * nb + 1], a, bq[2], bq[3]);
            }
        }

        const int m_lo = tile * SC_BM + warp * 16 + (lane >> 2);
        if (PASS == 1) {
            const bool ok_lo = m_lo < l_M, ok_hi = m_lo + 8 < l_M;
#pragma unroll
            for (int nb = 0; nb < SC_BN / 8; ++nb) {
                if (ok_lo) {
                    colv[nb][0] = fmaxf(colv[nb][0], acc[nb][0]);
                    colv[nb][1] = fmaxf(colv[nb][1], acc[nb][1]);
                }
                if (ok_hi) {
                    colv[nb][0] = fmaxf(colv[nb][0], acc[nb][2]);
                    colv[nb][1] = fmaxf(colv[nb][1], acc[nb][3]);
                }
            }
        } else {
            float v_lo = -INFINITY, v_hi = -INFINITY;
#pragma unroll
            for (int nb = 0; nb < SC_BN / 8; ++nb) {
                v_lo = fmaxf(v_lo, fmaxf(acc[nb][0] - colv[nb][0], acc[nb][1] - colv[nb][1]));
                v_hi = fmaxf(v_hi, fmaxf(acc[nb][2] - colv[nb][0], acc[nb][3] - colv[nb][1]));
            }
            v_lo = fmaxf(v_lo, __shfl_xor_sync(0xffffffffu, v_lo, 1));
            v_lo = fmaxf(v_lo, __shfl_xor_sync(0xffffffffu, v_lo, 2));
            v_hi = fmaxf(v_hi, __shfl_xor_sync(0xffffffffu, v_hi, 1));
            v_hi = fmaxf(v_hi, __shfl_xor_sync(0xffffffffu, v_hi, 2));
            if ((lane & 3) == 0) {
                uint32_t* out = p.skey + (int64_t)b * p.max_tokens;
                if (m_lo < l_M) atomicMax(out + m_lo, f32_to_key(v_lo));
                if (m_lo + 8 < l_M) atomicMax(out + m_lo + 8, f32_to_key(v_hi));
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();

    if (PASS == 1) {
        // column maxima: across the 8 row-lanes of the warp, then across warps
#pragma unroll
        for (int nb = 0; nb < SC_BN / 8; ++nb) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = colv[nb][e];
                v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
                v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
                v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
                if (lane < 4) sR[warp * SC_BN + nb * 8 + lane * 2 + e] = v;
            }
        }
        __syncthreads();
        for (int i = tid; i < SC_BN; i += SC_THREADS) {
            float v = sR[i];
#pragma unroll
            for (int w = 1; w < SC_THREADS / 32; ++w) v = fmaxf(v, sR[w * SC_BN + i]);
            if (q0 + i < p.l_C && v > -INFINITY) atomicMax(p.rkey + (int64_t)b * p.l_C + q0 + i, f32_to_key(v));
        }
    }
}

// ---------------------------------------------------------------------------
// l_C = 1: S[m] = q' . k'_m as a streaming matrix-vector product, with the front half of the
// selection fused in.  With a single query, Eq. 4 is s_m = S_m - r (r = max_m S_m), and the
// proximity pooling of Eq. 8 commutes with subtracting r (x -> fl(x - r) is monotone), so the
// kernel pools the raw scores: P_j = max of S over [j - eps, j + eps] clipped to M.  It leaves
//   * pkey[m]  = order-preserving key of P_m,
//   * ghist0   = per-sequence histogram of the keys' top 11 bits (first radix digit of Eq. 2),
//   * rkey[b]  = key of r (atomic max),
// and the selection kernel finds the k-th largest P, maps the threshold through fl(. - r) and
// compacts on fl(P_m - r): exactly the set that selecting on s' would give, ties included.
// A CTA owns up to SD_TOKENS consecutive middle tokens (plus eps recomputed neighbours on each side),
// so the window maxima come from shared memory and the histogram is flushed once per CTA.
// ---------------------------------------------------------------------------
constexpr int SD_TOKENS = 2048;
constexpr int SD_HALO = 16;          // largest eps
constexpr int SD_THREADS = 256;
constexpr int SD_BINS = 2048;

struct ScoreDecodeParams {
    const __nv_bfloat16* kc;
    const __nv_bfloat16* qc;    // [B, DC]
    uint32_t* rkey;             // [B]
    uint32_t* pkey;             // [B, max_tokens] keys of the pooled raw scores
    uint32_t* ghist0;           // [B, SD_BINS], zero on entry
    int64_t max_tokens;
    int eps;
    int chunk;                  // middle tokens per CTA: a multiple of SD_THREADS, at most SD_TOKENS
    SeqMeta meta;
};

template <int DC>
__global__ void __launch_bounds__(SD_THREADS)
score_decode_kernel(ScoreDecodeParams p) {
    constexpr int LPR = DC / 8;         // lanes per key row (16 bytes each)
    constexpr int RPW = 32 / LPR;       // rows per warp access
    constexpr int UNROLL = 4;
    __shared__ float sS[SD_TOKENS + 2 * SD_HALO];
    __shared__ uint32_t shist[SD_BINS];
    __shared__ float smax[SD_THREADS / 32];
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int a = blockIdx.x * p.chunk;                // first middle token of this CTA
    if (a >= l_M) return;
    const int nb = min(p.chunk, l_M - a);
    const int eps = p.eps;
    const uint4* kc = reinterpret_cast<const uint4*>(p.kc + ((int64_t)b * p.max_tokens + i_end) * DC);
    for (int i = tid; i < SD_BINS; i += SD_THREADS) shist[i] = 0u;

    float q[8];
    {
        uint4 v = reinterpret_cast<const uint4*>(p.qc + (int64_t)b * DC)[lane % LPR];
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __bfloat1622float2(h[i]);
            q[2 * i] = f.x;
            q[2 * i + 1] = f.y;
        }
    }
    // scores of the tokens [lo, hi): this CTA's own and the neighbours its windows reach
    const int lo = max(0, a - eps), hi = min(l_M, a + nb + eps);
    const int sub = lane / LPR, part = lane % LPR;
    float vmax = -INFINITY;
    for (int base = lo + warp * (RPW * UNROLL); base < hi; base += (SD_THREADS / 32) * (RPW * UNROLL)) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int m = base + u * RPW + sub;
            v[u] = (m < hi) ? __ldg(kc + (int64_t)m * LPR + part) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v[u]);
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float2 f = __bfloat1622float2(h[i]);
                acc = fmaf(q[2 * i], f.x, acc);
                acc = fmaf(q[2 * i + 1], f.y, acc);
            }
#pragma unroll
            for (int o = LPR / 2; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            const int m = base + u * RPW + sub;
            if (m < hi) {
                if (part == 0) sS[m - (a - eps)] = acc;
                vmax = fmaxf(vmax, acc);
            }
        }
    }
    // window positions outside M never win
    for (int i = tid; i < nb + 2 * eps; i += SD_THREADS) {
        const int m = a - eps + i;
        if (m < 0 || m >= l_M) sS[i] = -INFINITY;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, o));
    if (lane == 0) smax[warp] = vmax;
    __syncthreads();
    if (tid == 0) {
        float v = smax[0];
        for (int w = 1; w < SD_THREADS / 32; ++w) v = fmaxf(v, smax[w]);
        if (v > -INFINITY) atomicMax(p.rkey + b, f32_to_key(v));
    }
    // Eq. 8 on the raw scores, keys, first radix digit
    uint32_t* pk = p.pkey + (int64_t)b * p.max_tokens + a;
    float best[SD_TOKENS / SD_THREADS];
#pragma unroll
    for (int qd = 0; qd < SD_TOKENS / SD_THREADS; ++qd) best[qd] = -INFINITY;
    for (int w = 0; w <= 2 * eps; ++w) {
#pragma unroll
        for (int qd = 0; qd < SD_TOKENS / SD_THREADS; ++qd) {
            const int i = min(qd * SD_THREADS + tid, nb - 1);          // clamped lanes are not stored
            best[qd] = fmaxf(best[qd], sS[i + w]);
        }
    }
#pragma unroll
    for (int qd = 0; qd < SD_TOKENS / SD_THREADS; ++qd) {
        const int i = qd * SD_THREADS + tid;
        const bool valid = i < nb;
        const uint32_t key = f32_to_key(best[qd]);
        if (valid) pk[i] = key;
        // aggregated over the warp: neighbouring tokens crowd into a few bins
        const uint32_t peers = __match_any_sync(0xffffffffu, valid ? (key >> 21) : 0xffffffffu);
        if (valid && lane == __ffs(peers) - 1) atomicAdd(&shist[key >> 21], (uint32_t)__popc(peers));
    }
    __syncthreads();
    uint32_t* gh = p.ghist0 + (int64_t)b * SD_BINS;
    for (int i = tid; i < SD_BINS; i += SD_THREADS) {
        const uint32_t c = shist[i];
        if (c) atomicAdd(gh + i, c);
    }
}

template <int DC>
static cudaError_t launch_score_t(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache,
                                  const SeqMeta& meta, int max_lM, bool rkey_cleared, bool ghist_cleared, cudaStream_t st,
                                  bool* pooled_ready) {
    cudaError_t e = cudaSuccess;
    *pooled_ready = false;
    if (!rkey_cleared) e = cudaMemsetAsync(ctx->rkey, 0, sizeof(uint32_t) * (size_t)B * l_C, st);
    if (e != cudaSuccess) return e;
    if (l_C == 1) {
        ScoreDecodeParams p;
        p.kc = kc_cache; p.qc = ctx->Qc; p.rkey = ctx->rkey;
        p.pkey = ctx->pkey; p.ghist0 = ctx->ghist0;
        p.max_tokens = ctx->cfg.max_tokens; p.eps = ctx->cfg.eps; p.meta = meta;
        if (!ghist_cleared) {
            e = cudaMemsetAsync(ctx->ghist0, 0, sizeof(uint32_t) * (size_t)B * SD_BINS, st);
            if (e != cudaSuccess) return e;
        }
        // Tokens per CTA.  All CTAs are resident at once and the kernel ends with the SM that got the most work,
        // so the choice minimises (CTAs on the fullest SM) x (tokens per CTA + the CTA's serial start and tail:
        // clear, pooling, flush, worth about 256 tokens of loads).  Measured with 8 x 129k tokens: 2048 tokens
        // per CTA (504 CTAs, four on some SMs and three on others) 55 us, 1792 (576 CTAs, four nearly everywhere)
        // 52 us, 1536 (672 CTAs, five on some SMs) 71 us.
        int64_t chunk = SD_THREADS, best_cost = -1;
        for (int64_t c = SD_THREADS; c <= SD_TOKENS; c += SD_THREADS) {
            const int64_t n_ctas = (int64_t)B * ((max_lM + c - 1) / c);
            const int64_t cost = ((n_ctas + ctx->num_sms - 1) / ctx->num_sms) * (c + SD_THREADS);
            if (best_cost < 0 || cost <= best_cost) { best_cost = cost; chunk = c; }
        }
        p.chunk = (int)chunk;
        int gx = (max_lM + p.chunk - 1) / p.chunk;
        if (gx < 1) gx = 1;
        ProfScope prof(ctx, KC_SCORE_DECODE, st);
        e = launch_pdl(score_decode_kernel<DC>, dim3(gx, B), dim3(SD_THREADS), 0, st, p);
        ctx->launches += 1;
        *pooled_ready = true;
        return e;
    }
    // prefill-sized chunks with d' of 64 or 128: tcgen05 + TMA kernels (they clear what they accumulate into)
    if (score_uses_tc(ctx, B, l_C)) {
        e = launch_score_tc(ctx, B, l_C, kc_cache, meta, max_lM, st, pooled_ready);
        if (e != cudaErrorNotSupported) return e;
        cudaGetLastError();
    }
    // the pooling kernel that follows adds to the first-digit histograms
    e = cudaMemsetAsync(ctx->ghist0, 0, sizeof(uint32_t) * (size_t)B * SD_BINS, st);
    if (e != cudaSuccess) return e;
    e = cudaMemset2DAsync(ctx->skey, sizeof(uint32_t) * ctx->cfg.max_tokens, 0,
                          sizeof(uint32_t) * (size_t)max_lM, B, st);
    if (e != cudaSuccess) return e;
    ScoreParams p;
    p.kc = kc_cache; p.qc = ctx->Qc; p.rkey = ctx->rkey; p.skey = ctx->skey;
    p.max_tokens = ctx->cfg.max_tokens; p.l_C = l_C; p.meta = meta;
    const int qblocks = (l_C + SC_BN - 1) / SC_BN;
    const int n_tiles = (max_lM + SC_BM - 1) / SC_BM;
    int gx = (ctx->num_sms + qblocks * B - 1) / (qblocks * B);
    if (gx > n_tiles) gx = n_tiles;
    if (gx < 1) gx = 1;
    constexpr int smem = (SC_BN + SC_STAGES * SC_BM) * (DC / 8) * 16 + 8 * SC_BN * 4;
    e = cudaFuncSetAttribute(score_pass_kernel<DC, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_pass_kernel<DC, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(gx, qblocks, B);
    ProfScope prof(ctx, KC_SCORE_MMA, st);
    score_pass_kernel<DC, 1><<<grid, SC_THREADS, smem, st>>>(p);
    score_pass_kernel<DC, 2><<<grid, SC_THREADS, smem, st>>>(p);
    ctx->launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_score(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache, const SeqMeta& meta,
                         int max_lM, bool rkey_cleared, bool ghist_cleared, cudaStream_t st, bool* pooled_ready) {
    switch (ctx->dc) {
        case 32: return launch_score_t<32>(ctx, B, l_C, kc_cache, meta, max_lM, rkey_cleared, ghist_cleared, st, pooled_ready);
        case 64: return launch_score_t<64>(ctx, B, l_C, kc_cache, meta, max_lM, rkey_cleared, ghist_cleared, st, pooled_ready);
        case 128: return launch_score_t<128>(ctx, B, l_C, kc_cache, meta, max_lM, rkey_cleared, ghist_cleared, st, pooled_ready);
    }
    return cudaErrorInvalidValue;
}

}  // namespace esa
