// Eq. 3 + Eq. 4 on the full-dimension queries and keys (no compression), and the per-head vote of
// Section 4.3 -- the two scoring variants the paper compares its compressed scores against.
//
//   uniform    f_s(m; c) = sum_h q_{h,c} . k_{h,m}          (Eq. 3; head h reads key/value head h / G)
//              s_m = max_c ( f_s(m; c) - max_m' f_s(m'; c) )  (Eq. 4)
//   per head   every head h scores by itself, s_m^h = max_c ( q_{h,c} . k_{h,m} - max_m' q_{h,c} . k_{h,m'} ),
//              and s_m = max_h s_m^h
//
// Same two-pass scheme as the compressed scores (pass 1: the row maxima; pass 2: the scores again,
// minus the row maximum, maximum over the queries), on mma.sync tensor-core instructions: a CTA
// owns 128 keys x 128 queries, walks the heads of its slice with the accumulator in registers
// (uniform: all H heads summed into one accumulator; per head: one head per slice, blockIdx.z),
// and streams the per-head 128 x d operand tiles through double-buffered shared memory.  Both
// passes issue the same instruction sequence, so pass 2 reproduces pass 1's values bit for bit
// and the score of each query's arg-max is exactly 0.  The unpooled keys go to ctx->skey by
// atomic maximum (over query blocks and, per head, over heads); pooling and selection follow in
// the kernels of esa_select.cu.
#include "esa_internal.h"

namespace esa {

namespace {

constexpr int SF_BM = 128;      // keys per tile (8 warps x 16)
constexpr int SF_BN = 128;      // queries per CTA
constexpr int SF_THREADS = 256;

struct ScoreFullParams {
    const __nv_bfloat16* Q;     // [B, l_C, H, D]
    const __nv_bfloat16* K;     // [B, max_tokens, HG, D]
    uint32_t* rkey;             // [B, n_slices, l_C] ordered keys of the row maxima
    uint32_t* skey;             // [B, max_tokens] (index = m - i_end), zero on entry to pass 2
    int64_t max_tokens;
    int l_C, H, HG, G;
    int heads_per_slice;        // H (uniform) or 1 (per head)
    int n_slices;               // 1 or H
    SeqMeta meta;
};

template <int D, int PASS>
__global__ void __launch_bounds__(SF_THREADS)
score_full_kernel(ScoreFullParams p) {
    constexpr int CH = D / 8;
    extern __shared__ uint4 smem[];
    uint4* sQ = smem;                                   // 2 x [SF_BN][CH]
    uint4* sK = smem + 2 * SF_BN * CH;                  // 2 x [SF_BM][CH]
    float* sR = reinterpret_cast<float*>(sK + 2 * SF_BM * CH);   // [8][SF_BN] (pass 1) / [SF_BN] (pass 2)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.z / p.n_slices, slice = blockIdx.z % p.n_slices;
    const int h0 = slice * p.heads_per_slice, hc = p.heads_per_slice;
    const int q0 = blockIdx.y * SF_BN;
    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int n_tiles = (l_M + SF_BM - 1) / SF_BM;
    if ((int)blockIdx.x >= n_tiles) return;
    const __nv_bfloat16* Kb = p.K + ((int64_t)b * p.max_tokens + i_end) * p.HG * D;
    const __nv_bfloat16* Qb = p.Q + (int64_t)b * p.l_C * p.H * D;
    uint32_t* rk = p.rkey + ((int64_t)b * p.n_slices + slice) * p.l_C;

    auto load_q = [&](int buf, int h) {
        uint4* dst = sQ + buf * SF_BN * CH;
        for (int i = tid; i < SF_BN * CH; i += SF_THREADS) {
            const int r = i / CH, c = i % CH;
            const bool ok = q0 + r < p.l_C;
            cp_async16(&dst[swz<CH>(r, c)], Qb + ((int64_t)(ok ? q0 + r : 0) * p.H + h) * D + c * 8, ok ? 16 : 0);
        }
    };
    auto load_k = [&](int buf, int tile, int g) {
        uint4* dst = sK + buf * SF_BM * CH;
        const int m0 = tile * SF_BM;
        for (int i = tid; i < SF_BM * CH; i += SF_THREADS) {
            const int r = i / CH, c = i % CH;
            const bool ok = m0 + r < l_M;
            cp_async16(&dst[swz<CH>(r, c)], Kb + ((int64_t)(ok ? m0 + r : 0) * p.HG + g) * D + c * 8, ok ? 16 : 0);
        }
    };

    // r_c of this thread's query columns (pass 2) / running column maxima (pass 1)
    float colv[SF_BN / 8][2];
    if (PASS == 2) {
        for (int i = tid; i < SF_BN; i += SF_THREADS) sR[i] = (q0 + i < p.l_C) ? key_to_f32(rk[q0 + i]) : INFINITY;
        __syncthreads();
    }
#pragma unroll
    for (int nb = 0; nb < SF_BN / 8; ++nb) {
        colv[nb][0] = PASS == 2 ? sR[nb * 8 + (lane & 3) * 2] : -INFINITY;
        colv[nb][1] = PASS == 2 ? sR[nb * 8 + (lane & 3) * 2 + 1] : -INFINITY;
    }
    __syncthreads();

    // steps (tile, head) in order; the operands of step s + 1 are fetched while step s computes
    const int my_tiles = (n_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
    const int n_steps = my_tiles * hc;
    int kbuf = 0;                                       // buffer holding the K tile of the current step
    load_q(0, h0);
    load_k(0, blockIdx.x, h0 / p.G);
    cp_async_commit();
    float acc[SF_BN / 8][4];
    for (int s = 0; s < n_steps; ++s) {
        const int it = s / hc, i = s % hc;
        const int tile = blockIdx.x + it * gridDim.x;
        const int h = h0 + i;
        // prefetch the next step
        bool next_new_k = false;
        if (s + 1 < n_steps) {
            const int it2 = (s + 1) / hc, i2 = (s + 1) % hc;
            const int tile2 = blockIdx.x + it2 * gridDim.x, h2 = h0 + i2;
            load_q((s + 1) & 1, h2);
            next_new_k = tile2 != tile || h2 / p.G != h / p.G;
            if (next_new_k) load_k(kbuf ^ 1, tile2, h2 / p.G);
        }
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint4* tq = sQ + (s & 1) * SF_BN * CH;
        const uint4* tk = sK + kbuf * SF_BM * CH;
        if (i == 0) {
#pragma unroll
            for (int a = 0; a < SF_BN / 8; ++a)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[a][j] = 0.f;
        }
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t a[4];
            load_a_frag<CH>(a, tk, warp * 16, ks * 2, lane);
#pragma unroll
            for (int nb = 0; nb < SF_BN / 16; ++nb) {
                uint32_t bq[4];
                load_b_frag_nk<CH>(bq, tq, nb * 16, ks * 2, lane);
                mma_bf16_16816(acc[2 * nb], a, bq[0], bq[1]);
                mma_bf16_16816(acc[2 * nb + 1], a, bq[2], bq[3]);
            }
        }
        if (i == hc - 1) {
            const int m_lo = tile * SF_BM + warp * 16 + (lane >> 2);
            if (PASS == 1) {
                const bool ok_lo = m_lo < l_M, ok_hi = m_lo + 8 < l_M;
#pragma unroll
                for (int nb = 0; nb < SF_BN / 8; ++nb) {
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
                for (int nb = 0; nb < SF_BN / 8; ++nb) {
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
        }
        if (next_new_k) kbuf ^= 1;
        __syncthreads();
    }
    cp_async_wait<0>();

    if (PASS == 1) {
        // column maxima: across the 8 row-lanes of the warp, then across warps
#pragma unroll
        for (int nb = 0; nb < SF_BN / 8; ++nb) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = colv[nb][e];
                v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
                v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
                v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
                if (lane < 4) sR[warp * SF_BN + nb * 8 + lane * 2 + e] = v;
            }
        }
        __syncthreads();
        for (int i = tid; i < SF_BN; i += SF_THREADS) {
            float v = sR[i];
#pragma unroll
            for (int w = 1; w < SF_THREADS / 32; ++w) v = fmaxf(v, sR[w * SF_BN + i]);
            if (q0 + i < p.l_C && v > -INFINITY) atomicMax(rk + q0 + i, f32_to_key(v));
        }
    }
}

template <int D>
cudaError_t launch_full_t(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* K, const SeqMeta& meta,
                          int max_lM, bool per_head, cudaStream_t st) {
    ScoreFullParams p;
    p.Q = Q; p.K = K; p.rkey = ctx->rkey_heads; p.skey = ctx->skey;
    p.max_tokens = ctx->cfg.max_tokens; p.l_C = l_C; p.H = ctx->H; p.HG = ctx->HG; p.G = ctx->G;
    p.heads_per_slice = per_head ? 1 : ctx->H;
    p.n_slices = per_head ? ctx->H : 1;
    p.meta = meta;
    cudaError_t e = cudaMemsetAsync(ctx->rkey_heads, 0, sizeof(uint32_t) * (size_t)B * p.n_slices * l_C, st);
    if (e != cudaSuccess) return e;
    e = cudaMemset2DAsync(ctx->skey, sizeof(uint32_t) * ctx->cfg.max_tokens, 0, sizeof(uint32_t) * (size_t)max_lM, B, st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(ctx->ghist0, 0, sizeof(uint32_t) * (size_t)B * 2048, st);
    if (e != cudaSuccess) return e;
    constexpr int smem = 4 * 128 * (D / 8) * 16 + 8 * SF_BN * 4;
    e = cudaFuncSetAttribute(score_full_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_full_kernel<D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const int qblocks = (l_C + SF_BN - 1) / SF_BN;
    const int n_tiles = (max_lM + SF_BM - 1) / SF_BM;
    const int zs = B * p.n_slices;
    int gx = (2 * ctx->num_sms + qblocks * zs - 1) / (qblocks * zs);
    if (gx > n_tiles) gx = n_tiles;
    if (gx < 1) gx = 1;
    const dim3 grid(gx, qblocks, zs);
    ProfScope prof(ctx, KC_SCORE_FULL, st);
    score_full_kernel<D, 1><<<grid, SF_THREADS, smem, st>>>(p);
    score_full_kernel<D, 2><<<grid, SF_THREADS, smem, st>>>(p);
    ctx->launches += 2;
    return cudaGetLastError();
}

}  // namespace

// Fills ctx->skey with the unpooled full-dimension scores (ordered keys) and zeroes ctx->ghist0.
cudaError_t launch_score_full(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* Q, const __nv_bfloat16* K, const SeqMeta& meta,
                              int max_lM, bool per_head, cudaStream_t st) {
    if (ctx->d == 128) return launch_full_t<128>(ctx, B, l_C, Q, K, meta, max_lM, per_head, st);
    if (ctx->d == 64) return launch_full_t<64>(ctx, B, l_C, Q, K, meta, max_lM, per_head, st);
    return cudaErrorInvalidValue;
}

}  // namespace esa
