// Eq. 6 + Eq. 4 for prefill-sized chunks on the 5th-generation tensor cores.
//
//   S[c, m] = q'_c . k'_m          r_c = max_m S[c, m]          s_m = max_c ( S[c, m] - r_c )
//
// Two launches stream the compressed keys of the middle tokens through a TMA-fed ring of
// 128-key tiles; the chunk's compressed queries stay in shared memory.  S lives only in
// tensor memory (two accumulator buffers, so the epilogue of one tile overlaps the MMAs of
// the next):
//   pass 1  queries on the M side (TMEM lanes), keys on the N side: a thread owns one query
//           and folds the row maximum r_c over every tile in registers;
//   pass 2  keys on the M side, queries on the N side: a thread owns one key, subtracts the
//           r_c of every query column (read from shared memory) and keeps the maximum.
// Swapping the operands keeps both reductions inside a thread.  Every S[c, m] is the same
// sum of the same exact bf16 products taken in the same order over d' in both passes, so
// pass 2 reproduces pass 1's value and S - r_c is exactly 0 at each query's arg-max.
//
// Warp roles: warp 0 issues the TMA loads, warp 1 issues the MMAs (converged, lane 0
// leads), warps 2-5 run the epilogue (one TMEM lane quarter each).
#include "esa_internal.h"
#include "esa_umma.cuh"

namespace esa {

namespace {

constexpr int ST_KEYS = 128;       // keys per streamed tile
constexpr int ST_STAGES = 4;
constexpr int ST_THREADS = 192;

struct ScoreTcParams {
    uint32_t* rkey;     // [B, l_C] ordered keys of r_c
    uint32_t* skey;     // [B, max_tokens] ordered keys of s_m (index = m - i_end)
    int* status;
    int64_t max_tokens;
    int l_C;
    int combine;        // pass 2: more than one query block contributes to a key (atomic max)
    int clear_skey;     // pass 1: the CTAs of query block 0 zero skey for the tiles they visit
    SeqMeta meta;
};

enum { SB_Q_FULL = 0, SB_FULL = 1, SB_EMPTY = SB_FULL + ST_STAGES, SB_ACC_FULL = SB_EMPTY + ST_STAGES,
       SB_ACC_EMPTY = SB_ACC_FULL + 2, SB_COUNT = SB_ACC_EMPTY + 2 };

__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

template <int DC, int PASS>
__global__ void __launch_bounds__(ST_THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap qmap, ScoreTcParams p) {
    constexpr int NBLK = DC / 64;                        // 64-column blocks of a row
    constexpr int QROWS = PASS == 1 ? 128 : 256;         // queries of this CTA
    constexpr int TILE_BYTES = ST_KEYS * DC * 2;
    constexpr int Q_BYTES = QROWS * DC * 2;
    constexpr int ACC_COLS = PASS == 1 ? ST_KEYS : QROWS;   // accumulator columns per buffer
    constexpr int TMEM_COLS = 2 * ACC_COLS;

    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + Q_BYTES;
    float* sR = reinterpret_cast<float*>(sK + ST_STAGES * TILE_BYTES);      // [QROWS], pass 2
    __shared__ uint64_t bars[SB_COUNT];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int b = blockIdx.z;
    const int q0 = blockIdx.y * QROWS;
    const int i_end = p.meta.i_end[b];
    const int l_M = p.meta.m_end[b] - i_end;
    const int n_tiles = (l_M + ST_KEYS - 1) / ST_KEYS;
    // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
    const int my_tiles = (int)blockIdx.x < n_tiles ? (n_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    WaitCtx wc{&abort_flag, p.status};
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar(SB_Q_FULL), 1);
        for (int s = 0; s < ST_STAGES; ++s) {
            mbar_init(bar(SB_FULL + s), 1);
            mbar_init(bar(SB_EMPTY + s), 1);
        }
        for (int u = 0; u < 2; ++u) {
            mbar_init(bar(SB_ACC_FULL + u), 1);
            mbar_init(bar(SB_ACC_EMPTY + u), 128);
        }
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0 && my_tiles > 0) {
            tma_prefetch_desc(&kmap);
            tma_prefetch_desc(&qmap);
            mbar_arrive_expect_tx(bar(SB_Q_FULL), Q_BYTES);
#pragma unroll
            for (int blk = 0; blk < NBLK; ++blk)
#pragma unroll
                for (int r0 = 0; r0 < QROWS; r0 += 128)
                    tma_load_2d(smem_u32(sQ + blk * (QROWS * 128) + r0 * 128), &qmap, blk * 64, b * p.l_C + q0 + r0,
                                bar(SB_Q_FULL));
            const int64_t row_base = (int64_t)b * p.max_tokens + i_end;
            for (int i = 0; i < my_tiles; ++i) {
                const int s = i % ST_STAGES;
                const int tile = blockIdx.x + i * gridDim.x;
                mbar_wait(bar(SB_EMPTY + s), ((i / ST_STAGES) & 1) ^ 1, wc);
                mbar_arrive_expect_tx(bar(SB_FULL + s), TILE_BYTES);
#pragma unroll
                for (int blk = 0; blk < NBLK; ++blk)
                    tma_load_2d(smem_u32(sK + s * TILE_BYTES + blk * (ST_KEYS * 128)), &kmap, blk * 64,
                                (int)(row_base + (int64_t)tile * ST_KEYS), bar(SB_FULL + s));
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issue (converged warp, lane 0 leads)
        if (my_tiles > 0) {
            const uint32_t lead = lane == 0;
            const uint32_t hi = desc_hi_sw128();
            const uint32_t qlo = desc_lo_kmajor(smem_u32(sQ)), klo = desc_lo_kmajor(smem_u32(sK));
            constexpr uint32_t IDESC = idesc_bf16(128, ACC_COLS, false, false);
            mbar_wait(bar(SB_Q_FULL), 0, wc);
            for (int i = 0; i < my_tiles; ++i) {
                const int s = i % ST_STAGES, u = i & 1;
                mbar_wait(bar(SB_FULL + s), (i / ST_STAGES) & 1, wc);
                mbar_wait(bar(SB_ACC_EMPTY + u), ((i >> 1) & 1) ^ 1, wc);
                tc_fence_after_sync();
                const uint32_t k0 = klo + s * (TILE_BYTES >> 4);
                const uint32_t d = tmem + u * ACC_COLS;
#pragma unroll
                for (int ks = 0; ks < DC / 16; ++ks) {
                    const uint32_t oq = ((ks >> 2) * (QROWS * 128) + (ks & 3) * 32) >> 4;
                    const uint32_t ok = ((ks >> 2) * (ST_KEYS * 128) + (ks & 3) * 32) >> 4;
                    if (PASS == 1) umma_ss(d, qlo + oq, k0 + ok, hi, IDESC, ks, lead);     // S[c, m]
                    else umma_ss(d, k0 + ok, qlo + oq, hi, IDESC, ks, lead);               // S^T[m, c]
                }
                umma_commit(bar(SB_EMPTY + s), lead);
                umma_commit(bar(SB_ACC_FULL + u), lead);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: 4 warps, one TMEM lane quarter each
        const int quarter = warp & 3;
        const int et = (warp - 2) * 32 + lane;            // 0..127
        const uint32_t tbase = tmem_addr(tmem, quarter * 32, 0);
        if (PASS == 2) {
            for (int i = et; i < QROWS; i += 128)
                sR[i] = (q0 + i < p.l_C) ? key_to_f32(p.rkey[(int64_t)b * p.l_C + q0 + i]) : INFINITY;
            asm volatile("bar.sync 1, 128;\n" ::: "memory");
        }
        float rmax = -INFINITY;
        for (int i = 0; i < my_tiles; ++i) {
            const int u = i & 1;
            const int tile = blockIdx.x + i * gridDim.x;
            mbar_wait(bar(SB_ACC_FULL + u), (i >> 1) & 1, wc);
            tc_fence_after_sync();
            if (PASS == 1) {
                const int key0 = tile * ST_KEYS;
                const bool tail = key0 + ST_KEYS > l_M;
                if (p.clear_skey && blockIdx.y == 0 && key0 + et < l_M) p.skey[(int64_t)b * p.max_tokens + key0 + et] = 0u;
#pragma unroll
                for (int c0 = 0; c0 < ST_KEYS; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tbase + u * ACC_COLS + c0, v);
                    tmem_wait_ld();
                    if (tail) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (key0 + c0 + j >= l_M) v[j] = 0xff800000u;
                    }
                    float m0 = rmax, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        m0 = max3f(m0, __uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                        m1 = max3f(m1, __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                        m2 = max3f(m2, __uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                        m3 = max3f(m3, __uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                    }
                    rmax = fmaxf(max3f(m0, m1, m2), m3);
                }
            } else {
                float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY;
#pragma unroll
                for (int c0 = 0; c0 < QROWS; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tbase + u * ACC_COLS + c0, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        const float4 ra = *reinterpret_cast<const float4*>(sR + c0 + j);
                        const float4 rb = *reinterpret_cast<const float4*>(sR + c0 + j + 4);
                        a0 = max3f(a0, __uint_as_float(v[j]) - ra.x, __uint_as_float(v[j + 1]) - ra.y);
                        a1 = max3f(a1, __uint_as_float(v[j + 2]) - ra.z, __uint_as_float(v[j + 3]) - ra.w);
                        a2 = max3f(a2, __uint_as_float(v[j + 4]) - rb.x, __uint_as_float(v[j + 5]) - rb.y);
                        a3 = max3f(a3, __uint_as_float(v[j + 6]) - rb.z, __uint_as_float(v[j + 7]) - rb.w);
                    }
                }
                const float sm = fmaxf(max3f(a0, a1, a2), a3);
                const int m = tile * ST_KEYS + quarter * 32 + lane;
                if (m < l_M) {
                    uint32_t* out = p.skey + (int64_t)b * p.max_tokens + m;
                    if (p.combine) atomicMax(out, f32_to_key(sm));
                    else *out = f32_to_key(sm);
                }
            }
            tc_fence_before_sync();
            mbar_arrive(bar(SB_ACC_EMPTY + u));
        }
        if (PASS == 1) {
            const int q = q0 + quarter * 32 + lane;
            if (q < p.l_C && rmax > -INFINITY) atomicMax(p.rkey + (int64_t)b * p.l_C + q, f32_to_key(rmax));
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

template <int DC>
cudaError_t launch_t(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache, const SeqMeta& meta, int max_lM,
                     cudaStream_t st) {
    CUtensorMap kmap, qmap;
    if (!make_tensor_map_bf16(&kmap, kc_cache, (uint64_t)B * ctx->cfg.max_tokens, DC, 128)) return cudaErrorNotSupported;
    if (!make_tensor_map_bf16(&qmap, ctx->Qc, (uint64_t)B * l_C, DC, 128)) return cudaErrorNotSupported;
    ScoreTcParams p;
    p.rkey = ctx->rkey; p.skey = ctx->skey; p.status = ctx->status;
    p.max_tokens = ctx->cfg.max_tokens; p.l_C = l_C; p.meta = meta;
    const int n_tiles = (max_lM + ST_KEYS - 1) / ST_KEYS;
    constexpr int smem1 = 128 * DC * 2 + ST_STAGES * ST_KEYS * DC * 2 + 1024 + 1024;
    constexpr int smem2 = 256 * DC * 2 + ST_STAGES * ST_KEYS * DC * 2 + 1024 + 1024;
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<DC, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_tc_kernel<DC, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2);
    if (e != cudaSuccess) return e;
    auto grid_x = [&](int qblocks) {
        int gx = (ctx->num_sms + qblocks * B - 1) / (qblocks * B);
        if (gx > n_tiles) gx = n_tiles;
        return gx < 1 ? 1 : gx;
    };
    const int qb1 = (l_C + 127) / 128, qb2 = (l_C + 255) / 256;
    p.combine = 0;
    p.clear_skey = qb2 > 1;
    e = launch_pdl(score_tc_kernel<DC, 1>, dim3(grid_x(qb1), qb1, B), dim3(ST_THREADS), smem1, st, kmap, qmap, p);
    if (e != cudaSuccess) return e;
    p.combine = qb2 > 1;
    e = launch_pdl(score_tc_kernel<DC, 2>, dim3(grid_x(qb2), qb2, B), dim3(ST_THREADS), smem2, st, kmap, qmap, p);
    if (e != cudaSuccess) return e;
    ctx->launches += 2;
    return cudaGetLastError();
}

}  // namespace

// Both scoring passes for chunks of at least 64 queries and d' of 64 or 128; rkey must be zeroed.
// Returns cudaErrorNotSupported when this path does not cover the shape.
cudaError_t launch_score_tc(esa_ctx* ctx, int B, int l_C, const __nv_bfloat16* kc_cache, const SeqMeta& meta,
                            int max_lM, cudaStream_t st) {
    if (l_C < 64) return cudaErrorNotSupported;
    if (ctx->dc == 128) return launch_t<128>(ctx, B, l_C, kc_cache, meta, max_lM, st);
    if (ctx->dc == 64) return launch_t<64>(ctx, B, l_C, kc_cache, meta, max_lM, st);
    return cudaErrorNotSupported;
}

}  // namespace esa
