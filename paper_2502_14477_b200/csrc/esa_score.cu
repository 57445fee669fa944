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
// l_C = 1: S[m] = q' . k'_m as a streaming matrix-vector product.
// ---------------------------------------------------------------------------
struct ScoreDecodeParams {
    const __nv_bfloat16* kc;
    const __nv_bfloat16* qc;    // [B, DC]
    uint32_t* rkey;             // [B]
    float* sraw;                // [B, max_tokens]
    int64_t max_tokens;
    SeqMeta meta;
};

template <int DC>
__global__ void __launch_bounds__(256)
score_decode_kernel(ScoreDecodeParams p) {
    constexpr int LPR = DC / 8;         // lanes per key row (16 bytes each)
    constexpr int RPW = 32 / LPR;       // rows per warp access
    constexpr int UNROLL = 4;
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const uint4* kc = reinterpret_cast<const uint4*>(p.kc + ((int64_t)b * p.max_tokens + i_end) * DC);
    float* out = p.sraw + (int64_t)b * p.max_tokens;

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
    const int sub = lane / LPR, part = lane % LPR;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    float vmax = -INFINITY;
    for (int64_t base = warp_global * (RPW * UNROLL); base < l_M; base += n_warps * (RPW * UNROLL)) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            int64_t m = base + u * RPW + sub;
            v[u] = (m < l_M) ? __ldg(kc + m * LPR + part) : make_uint4(0, 0, 0, 0);
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
            int64_t m = base + u * RPW + sub;
            if (m < l_M) {
                if (part == 0) out[m] = acc;
                vmax = fmaxf(vmax, acc);
            }
        }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, o));
    __shared__ float smax[8];
    if (lane == 0) smax[threadIdx.x >> 5] = vmax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float v = smax[0];
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) v = fmaxf(v, smax[w]);
        if (v > -INFINITY) atomicMax(p.rkey + b, f32_to_key(v));
    }
}

template <int DC>
static cudaError_t launch_score_t(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache,
                                  const SeqMeta& meta, int max_lM, bool rkey_cleared, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
    if (!rkey_cleared) e = cudaMemsetAsync(ctx->rkey, 0, sizeof(uint32_t) * (size_t)B * l_C, st);
    if (e != cudaSuccess) return e;
    if (l_C == 1) {
        ScoreDecodeParams p;
        p.kc = kc_cache; p.qc = ctx->Qc; p.rkey = ctx->rkey;
        p.sraw = reinterpret_cast<float*>(ctx->skey);
        p.max_tokens = ctx->cfg.max_tokens; p.meta = meta;
        constexpr int rows_per_block = 8 * (32 / (DC / 8)) * 4;
        int gx = (max_lM + rows_per_block - 1) / rows_per_block;
        int cap = (8 * ctx->num_sms + B - 1) / B;
        if (gx > cap) gx = cap;
        if (gx < 1) gx = 1;
        e = launch_pdl(score_decode_kernel<DC>, dim3(gx, B), dim3(256), 0, st, p);
        ctx->launches += 1;
        return e;
    }
    // prefill-sized chunks with d' of 64 or 128: tcgen05 + TMA kernels (they clear skey themselves)
    if (score_uses_tc(ctx, B, l_C)) {
        e = launch_score_tc(ctx, B, l_C, kc_cache, meta, max_lM, st);
        if (e != cudaErrorNotSupported) return e;
        cudaGetLastError();
    }
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
    score_pass_kernel<DC, 1><<<grid, SC_THREADS, smem, st>>>(p);
    score_pass_kernel<DC, 2><<<grid, SC_THREADS, smem, st>>>(p);
    ctx->launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_score(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache, const SeqMeta& meta,
                         int max_lM, bool rkey_cleared, cudaStream_t st) {
    switch (ctx->dc) {
        case 32: return launch_score_t<32>(ctx, B, l_C, kc_cache, meta, max_lM, rkey_cleared, st);
        case 64: return launch_score_t<64>(ctx, B, l_C, kc_cache, meta, max_lM, rkey_cleared, st);
        case 128: return launch_score_t<128>(ctx, B, l_C, kc_cache, meta, max_lM, rkey_cleared, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace esa
